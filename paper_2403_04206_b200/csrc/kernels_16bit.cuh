// 16-bit storage (bfloat16 / half) variants of the two streaming kernels: parameters, gradients
// and centre are stored in T, all arithmetic is the fp32 / fp64 arithmetic of the fp32 kernels, and
// results are rounded to nearest-even once, on the store.  Half the bytes per element.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kernels.cuh"

namespace grawa {

// Conversions between a 32-bit word holding two T and two floats.
template <typename T> struct Pair16;
template <> struct Pair16<__nv_bfloat16> {
    static __device__ __forceinline__ void unpack(unsigned w, float& lo, float& hi)
    {
        lo = __uint_as_float(w << 16);              // a bfloat16 is the upper half of a float
        hi = __uint_as_float(w & 0xffff0000u);
    }
    static __device__ __forceinline__ unsigned pack(float lo, float hi)
    {
        const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<const unsigned*>(&v);
    }
    // lo += w.lo^2, hi += w.hi^2: fused multiply-add with 16-bit sources and an fp32 accumulator (the
    // sources are widened exactly, one rounding: the value of fmaf on the unpacked elements)
    static __device__ __forceinline__ void square_add(unsigned w, float& lo, float& hi)
    {
        asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tfma.rn.f32.bf16 %0, l, l, %0;\n\tfma.rn.f32.bf16 %1, h, h, %1;\n\t}"
            : "+f"(lo), "+f"(hi) : "r"(w));
    }
    static __device__ __forceinline__ float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};
template <> struct Pair16<__half> {
    static __device__ __forceinline__ void unpack(unsigned w, float& lo, float& hi)
    {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
        lo = f.x;
        hi = f.y;
    }
    static __device__ __forceinline__ unsigned pack(float lo, float hi)
    {
        const __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<const unsigned*>(&v);
    }
    static __device__ __forceinline__ void square_add(unsigned w, float& lo, float& hi)
    {
        asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tfma.rn.f32.f16 %0, l, l, %0;\n\tfma.rn.f32.f16 %1, h, h, %1;\n\t}"
            : "+f"(lo), "+f"(hi) : "r"(w));
    }
    static __device__ __forceinline__ float load1(const __half* p) { return __half2float(*p); }
    static __device__ __forceinline__ void store1(__half* p, float v) { *p = __float2half_rn(v); }
};

// Eight consecutive elements travel as one 16-byte word and stay packed in registers (four
// registers instead of eight) until the arithmetic needs them.
template <typename T>
__device__ __forceinline__ void unpack8(const uint4& r, float (&o)[8])
{
    Pair16<T>::unpack(r.x, o[0], o[1]); Pair16<T>::unpack(r.y, o[2], o[3]);
    Pair16<T>::unpack(r.z, o[4], o[5]); Pair16<T>::unpack(r.w, o[6], o[7]);
}
template <typename T>
__device__ __forceinline__ uint4 pack8(const float (&o)[8])
{
    uint4 r;
    r.x = Pair16<T>::pack(o[0], o[1]); r.y = Pair16<T>::pack(o[2], o[3]);
    r.z = Pair16<T>::pack(o[4], o[5]); r.w = Pair16<T>::pack(o[6], o[7]);
    return r;
}

// [b, e) -> scalar head, body aligned to 8 elements (16 bytes), scalar tail.
__device__ __forceinline__ void split_range16(long long b, long long e, int vec_ok, long long& hb, long long& te)
{
    if (vec_ok) {
        hb = min((b + 7) & ~7LL, e);
        te = max(e & ~7LL, hb);
    } else {
        hb = e;
        te = e;
    }
}

// Step 1 on 16-bit gradients: same work list, same fp32-run / fp64-combine scheme as sumsq_kernel;
// a thread's 16-byte load carries 8 elements, each with its own fp32 accumulator.  Six CTAs per SM
// (40 registers) like the fp32 kernel: measured 4 % faster than five on the ViT-B/16 table.
template <typename T, int UNROLL>
__global__ void __launch_bounds__(kThreads, 6)
sumsq16_kernel(const __grid_constant__ ConstPtrs grads, StepScratch sc, int items, int vec_ok)
{
    __shared__ double warp_part[2][kThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int C = sc.C;
    // the work list belongs to the plan, not to the kernel before this one: fetch the first item early
    Segment first_sg = Segment{0, 0, 0};
    if (static_cast<int>(blockIdx.x) < items) first_sg = sc.segs[blockIdx.x % C];
    // L2 hints for the items further on, on short problems (see sumsq_kernel)
    if (static_cast<int>(blockIdx.x) < sc.prefetch_stride && tid < sc.prefetch_waves) {
        const long long it = blockIdx.x + static_cast<long long>(tid + 1) * sc.prefetch_stride;
        if (it < items) {
            const int pm = static_cast<int>(it / C);
            const Segment sg = sc.segs[it - static_cast<long long>(pm) * C];
            long long phb, pte;
            split_range16(sg.begin, sg.begin + sg.len, vec_ok, phb, pte);
            const unsigned bytes = static_cast<unsigned>(pte - phb) * 2u;         // a multiple of 16
            if (bytes > 0 && in_bounds(phb, pte - phb, sg.begin, sg.begin + sg.len, sc.n))
                prefetch_l2(reinterpret_cast<const T*>(grads.p[pm]) + phb, bytes);
        }
    }
    grid_dependency_sync();
    // Which copy of the digit rows to add into: needed only by thread 0 when an item is done, and by
    // everybody after the last item; thread 0 fetches it now and hands it on through shared memory,
    // so that no thread waits for it in front of its gradient loads.
    __shared__ int buf_sm;
    int buf = 0;
    if (tid == 0) buf = __ldcg(sc.next_buf);

    int parity = 0;
    for (int item = blockIdx.x; item < items; item += gridDim.x, parity ^= 1) {
        const int m = item / C;
        const int s = item - m * C;
        const Segment sg = (item == static_cast<int>(blockIdx.x)) ? first_sg : sc.segs[s];
        const T* __restrict__ g = reinterpret_cast<const T*>(grads.p[m]);
        const long long b = sg.begin, e = b + sg.len;
        long long hb, te;
        split_range16(b, e, vec_ok, hb, te);
        double dacc = 0.0;

        const int ncol = static_cast<int>((te - hb) >> 3);
        const uint4* __restrict__ g8 = reinterpret_cast<const uint4*>(g + hb);
        for (int c0 = 0; c0 < ncol; c0 += kThreads * UNROLL) {
            uint4 raw[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int c = c0 + u * kThreads + tid;
                raw[u] = (c < ncol && in_bounds(hb + 8LL * c, 8, b, e, sc.n)) ? __ldcs(g8 + c) : make_uint4(0u, 0u, 0u, 0u);      // all-zero bits are 0.0 in both types
            }
            float a[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) a[t] = 0.f;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                Pair16<T>::square_add(raw[u].x, a[0], a[1]);
                Pair16<T>::square_add(raw[u].y, a[2], a[3]);
                Pair16<T>::square_add(raw[u].z, a[4], a[5]);
                Pair16<T>::square_add(raw[u].w, a[6], a[7]);
            }
            dacc += ((static_cast<double>(a[0]) + static_cast<double>(a[1])) + (static_cast<double>(a[2]) + static_cast<double>(a[3]))) +
                    ((static_cast<double>(a[4]) + static_cast<double>(a[5])) + (static_cast<double>(a[6]) + static_cast<double>(a[7])));
        }
        for (long long i = b + tid; i < hb; i += kThreads) {
            const double v = in_bounds(i, 1, b, e, sc.n) ? static_cast<double>(Pair16<T>::load1(g + i)) : 0.0;
            dacc += v * v;
        }
        for (long long i = te + tid; i < e; i += kThreads) {
            const double v = in_bounds(i, 1, b, e, sc.n) ? static_cast<double>(Pair16<T>::load1(g + i)) : 0.0;
            dacc += v * v;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) dacc += __shfl_down_sync(0xffffffffu, dacc, d);
        if (lane == 0) warp_part[parity][warp] = dacc;
        if (tid == 0) buf_sm = buf;
        __syncthreads();
        if (tid == 0) {
            double total = 0.0;
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) total += warp_part[parity][w];
            unsigned long long* bins = sc.bins + static_cast<size_t>(buf) * bins_copy_words(sc);
            if (scratch_ok(buf, 2) && scratch_ok(static_cast<long long>(sg.layer) * sc.M + m, static_cast<long long>(sc.K) * sc.M))
                bins_add(bins + static_cast<size_t>(sg.layer) * sc.M + m, static_cast<size_t>(sc.K) * sc.M, total);
        }
    }
    bins_turnover(sc, buf_sm);           // every CTA has had at least one item, hence one barrier after the write
}

// Shape of the 16-bit centre+pull kernel: columns of WORDS 32-bit words (two elements each) kept
// packed in registers: 16-byte columns up to 8 workers, 8-byte columns above.  Up to 4 workers a
// thread has as many columns in flight as the fp32 kernel (the same bytes in flight, a CTA covers
// twice the elements per pass: measured 5 % faster on the VGG-16 table); above that one column,
// because two need more than 128 registers (measured: slower at M = 8, no faster at M = 16).  The
// work lists of 16-bit plans are cut with this pass size.
__host__ __device__ constexpr int pull16_words(int M) { return (M <= 8) ? 4 : 2; }
__host__ __device__ constexpr int pull16_cols(int M) { return (M <= 2) ? 8 : (M <= 4) ? 4 : 1; }
__host__ __device__ constexpr int pull16_pass_elems(int M) { return kThreads * pull16_cols(M) * pull16_words(M) * 2; }

template <int WORDS> struct Words;
template <> struct Words<4> {
    static __device__ __forceinline__ void ld(const void* p, unsigned (&o)[4])
    {
        const uint4 r = __ldcs(reinterpret_cast<const uint4*>(p));
        o[0] = r.x; o[1] = r.y; o[2] = r.z; o[3] = r.w;
    }
    static __device__ __forceinline__ void st(void* p, const unsigned (&o)[4]) { __stcs(reinterpret_cast<uint4*>(p), make_uint4(o[0], o[1], o[2], o[3])); }
};
template <> struct Words<8> {                       // one 256-bit access; the address is 32-byte aligned
    static __device__ __forceinline__ void ld(const void* p, unsigned (&o)[8])
    {
        asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(o[0]), "=r"(o[1]), "=r"(o[2]), "=r"(o[3]), "=r"(o[4]), "=r"(o[5]), "=r"(o[6]), "=r"(o[7]) : "l"(p) : "memory");
    }
    static __device__ __forceinline__ void st(void* p, const unsigned (&o)[8])
    {
        asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     :: "l"(p), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
    }
};
template <> struct Words<2> {
    static __device__ __forceinline__ void ld(const void* p, unsigned (&o)[2])
    {
        const uint2 r = __ldcs(reinterpret_cast<const uint2*>(p));
        o[0] = r.x; o[1] = r.y;
    }
    static __device__ __forceinline__ void st(void* p, const unsigned (&o)[2]) { __stcs(reinterpret_cast<uint2*>(p), make_uint2(o[0], o[1])); }
};

template <typename T, int M>
__device__ __forceinline__ void pull16_scalar(const MutPtrs& x, T* center, const float* w, float lambda, float oml,
                                              long long i)
{
    float v[M];
#pragma unroll
    for (int m = 0; m < M; ++m) v[m] = Pair16<T>::load1(reinterpret_cast<const T*>(x.p[m]) + i);
    float c = w[0] * v[0];
#pragma unroll
    for (int m = 1; m < M; ++m) c = fmaf(w[m], v[m], c);
    if (center) Pair16<T>::store1(center + i, c);
#pragma unroll
    for (int m = 0; m < M; ++m) Pair16<T>::store1(reinterpret_cast<T*>(x.p[m]) + i, fmaf(lambda, c, oml * v[m]));
}

// Steps 4-5 on 16-bit parameters: same arithmetic as center_pull_kernel (fp32 FMA chain over
// m = 0..M-1, pull from the unrounded fp32 centre), one rounding on each store.
// WIDE (up to 4 workers, every base 32-byte aligned): 32-byte columns, half as many per thread.
template <typename T, int M, bool PER_LAYER, bool WIDE>
__global__ void __launch_bounds__(kThreads, 2)
center_pull16_kernel(MutPtrs x, T* __restrict__ center, const float* __restrict__ beta, const Segment* __restrict__ segs,
                     int item_begin, int item_end, long long n, int tile, float lambda, int vec_ok)
{
    static_assert(!WIDE || M <= 4, "32-byte columns are for up to 4 workers");
    Segment first_sg = Segment{0, 0, 0};           // plan data: independent of the kernel before this one
    if (PER_LAYER && item_begin + static_cast<int>(blockIdx.x) < item_end) first_sg = segs[item_begin + blockIdx.x];
    grid_dependency_sync();
    constexpr int COLS = WIDE ? pull16_cols(M) / 2 : pull16_cols(M);
    constexpr int WORDS = WIDE ? 8 : pull16_words(M);
    constexpr int VEC = 2 * WORDS;                 // elements per column
    const float oml = 1.0f - lambda;
    const int tid = threadIdx.x;
    float w[M];
    if (!PER_LAYER) {
#pragma unroll
        for (int m = 0; m < M; ++m) w[m] = beta[m];
    }
    for (int item = item_begin + blockIdx.x; item < item_end;) {
        long long b, e;
        if (PER_LAYER) {
            const Segment sg = first_sg;
            b = sg.begin;
            e = b + sg.len;
            const float* __restrict__ bt = beta + static_cast<size_t>(sg.layer) * M;
#pragma unroll
            for (int m = 0; m < M; ++m) w[m] = bt[m];
        } else {
            b = static_cast<long long>(item) * tile;
            e = min(n, b + tile);
        }
        long long hb = e, te = e;                                 // body aligned to a column (VEC is 4, 8 or 16 elements)
        if (vec_ok) {
            hb = min((b + (WIDE ? 15 : 7)) & ~static_cast<long long>(WIDE ? 15 : 7), e);
            te = max(e & ~static_cast<long long>(WIDE ? 15 : 7), hb);
        }
        const int ncol = static_cast<int>((te - hb) / VEC);      // te - hb is a multiple of 8 (16 when WIDE)
        for (int c0 = 0; c0 < ncol; c0 += kThreads * COLS) {
            unsigned raw[COLS][M][WORDS];
#pragma unroll
            for (int q = 0; q < COLS; ++q) {
                const int c = c0 + q * kThreads + tid;
                if (c < ncol && in_bounds(hb + static_cast<long long>(c) * VEC, VEC, b, e, n)) {
#pragma unroll
                    for (int m = 0; m < M; ++m)
                        Words<WORDS>::ld(reinterpret_cast<const T*>(x.p[m]) + hb + static_cast<long long>(c) * VEC, raw[q][m]);
                }
            }
#pragma unroll
            for (int q = 0; q < COLS; ++q) {
                const int c = c0 + q * kThreads + tid;
                if (c < ncol && in_bounds(hb + static_cast<long long>(c) * VEC, VEC, b, e, n)) {
                    // the column in pieces of at most 8 elements: centre (fp32 FMA chain over the workers),
                    // then the pulled workers packed back in place; stores of whole columns at the end
                    constexpr int HW = WORDS < 4 ? WORDS : 4;      // words per piece
                    unsigned oc[WORDS];
#pragma unroll
                    for (int h = 0; h < WORDS / HW; ++h) {
                        float cc[2 * HW];
#pragma unroll
                        for (int k = 0; k < HW; ++k) {
                            float lo, hi;
                            Pair16<T>::unpack(raw[q][0][h * HW + k], lo, hi);
                            cc[2 * k] = w[0] * lo;
                            cc[2 * k + 1] = w[0] * hi;
                        }
#pragma unroll
                        for (int m = 1; m < M; ++m) {
#pragma unroll
                            for (int k = 0; k < HW; ++k) {
                                float lo, hi;
                                Pair16<T>::unpack(raw[q][m][h * HW + k], lo, hi);
                                cc[2 * k] = fmaf(w[m], lo, cc[2 * k]);
                                cc[2 * k + 1] = fmaf(w[m], hi, cc[2 * k + 1]);
                            }
                        }
#pragma unroll
                        for (int k = 0; k < HW; ++k) oc[h * HW + k] = Pair16<T>::pack(cc[2 * k], cc[2 * k + 1]);
#pragma unroll
                        for (int m = 0; m < M; ++m) {
#pragma unroll
                            for (int k = 0; k < HW; ++k) {
                                float lo, hi;
                                Pair16<T>::unpack(raw[q][m][h * HW + k], lo, hi);
                                raw[q][m][h * HW + k] = Pair16<T>::pack(fmaf(lambda, cc[2 * k], oml * lo), fmaf(lambda, cc[2 * k + 1], oml * hi));
                            }
                        }
                    }
                    if (center) Words<WORDS>::st(center + hb + static_cast<long long>(c) * VEC, oc);
#pragma unroll
                    for (int m = 0; m < M; ++m) Words<WORDS>::st(reinterpret_cast<T*>(x.p[m]) + hb + static_cast<long long>(c) * VEC, raw[q][m]);
                }
            }
        }
        for (long long i = b + tid; i < hb; i += kThreads)
            if (in_bounds(i, 1, b, e, n)) pull16_scalar<T, M>(x, center, w, lambda, oml, i);
        for (long long i = te + tid; i < e; i += kThreads)
            if (in_bounds(i, 1, b, e, n)) pull16_scalar<T, M>(x, center, w, lambda, oml, i);
        item += gridDim.x;
        if (PER_LAYER && item < item_end) first_sg = segs[item];
    }
}

// Steps 4-5 on 16-bit parameters for 5..16 workers.  Sixteen 16-byte columns (the same bytes in flight
// as the fp32 kernel; two columns of up to eight workers) do not fit in registers next to their
// arithmetic, so every thread copies its columns of each worker straight from global to its own slots
// of shared memory with asynchronous
// 16-byte copies (`cp.async`, no registers held while they fly, L1 bypassed), waits for its own
// copies only (no CTA barrier: a thread reads nothing but what it copied), and then walks the
// workers twice from shared memory: the fp32 FMA chain of the centre, then the pull and one
// 16-byte store per worker.  Same arithmetic and rounding as center_pull16_kernel.  Shared memory:
// COLS x M x 256 x 16 bytes (64 KB at M = 16 and at M = 8), three CTAs per SM.
__host__ __device__ constexpr int pull16s_cols(int M) { return (M <= 8) ? 2 : 1; }     // 16-byte columns per thread in flight
__host__ __device__ constexpr int pull16s_pass_elems(int M) { return kThreads * 8 * pull16s_cols(M); }

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<unsigned>(__cvta_generic_to_shared(smem_dst))), "l"(gsrc)
                 : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

template <typename T, int M, bool PER_LAYER>
__global__ void __launch_bounds__(kThreads, 3)
center_pull16_staged_kernel(MutPtrs x, T* __restrict__ center, const float* __restrict__ beta, const Segment* __restrict__ segs,
                            int item_begin, int item_end, long long n, int tile, float lambda, int preload)
{
    extern __shared__ __align__(16) uint4 stage16[];          // [COLS][M][kThreads]
    constexpr int COLS = pull16s_cols(M);
    const int tid = threadIdx.x;
    int item = item_begin + blockIdx.x;
    int layer = 0, ncol = 0;
    long long b = 0, e = 0, hb = 0, te = 0;
    auto locate = [&](int it) {
        if (PER_LAYER) {
            const Segment sg = segs[it];
            b = sg.begin;
            e = b + sg.len;
            layer = sg.layer;
        } else {
            b = static_cast<long long>(it) * tile;
            e = min(n, b + tile);
        }
        split_range16(b, e, 1, hb, te);
        ncol = static_cast<int>((te - hb) >> 3);
    };
    auto fetch = [&](int c0) {                                  // this thread's columns of every worker -> shared memory
#pragma unroll
        for (int q = 0; q < COLS; ++q) {
            const int c = c0 + q * kThreads + tid;
            if (c < ncol && in_bounds(hb + 8LL * c, 8, b, e, n)) {
#pragma unroll
                for (int m = 0; m < M; ++m)
                    cp_async16(&stage16[(q * M + m) * kThreads + tid], reinterpret_cast<const T*>(x.p[m]) + hb + 8LL * c);
            }
        }
    };
    bool fetched = false;
    if (item < item_end) {
        locate(item);
        if (preload) {                                          // see center_pull_kernel for when this is valid
            fetch(0);
            fetched = true;
        }
    }
    grid_dependency_sync();
    const float oml = 1.0f - lambda;
    __shared__ float w[M];                                      // the item's weights, read where they are used
    while (item < item_end) {
        __syncthreads();                                        // nobody still reads the previous item's weights
        if (tid < M) w[tid] = PER_LAYER ? beta[static_cast<size_t>(layer) * M + tid] : beta[tid];
        __syncthreads();
        for (int c0 = 0; c0 < ncol; c0 += kThreads * COLS) {
            if (!fetched) fetch(c0);
            fetched = false;
            cp_async_wait_all();
#pragma unroll
            for (int q = 0; q < COLS; ++q) {
                const int c = c0 + q * kThreads + tid;
                if (c >= ncol || !in_bounds(hb + 8LL * c, 8, b, e, n)) continue;
                const uint4* col = stage16 + q * M * kThreads + tid;
                float cc[8];
                {
                    float v[8];
                    unpack8<T>(col[0], v);
#pragma unroll
                    for (int t = 0; t < 8; ++t) cc[t] = w[0] * v[t];
                }
#pragma unroll 4
                for (int m = 1; m < M; ++m) {
                    float v[8];
                    unpack8<T>(col[m * kThreads], v);
#pragma unroll
                    for (int t = 0; t < 8; ++t) cc[t] = fmaf(w[m], v[t], cc[t]);
                }
                if (center) __stcs(reinterpret_cast<uint4*>(center + hb) + c, pack8<T>(cc));
#pragma unroll 4
                for (int m = 0; m < M; ++m) {
                    float v[8];
                    unpack8<T>(col[m * kThreads], v);
#pragma unroll
                    for (int t = 0; t < 8; ++t) v[t] = fmaf(lambda, cc[t], oml * v[t]);
                    __stcs(reinterpret_cast<uint4*>(reinterpret_cast<T*>(x.p[m]) + hb) + c, pack8<T>(v));
                }
            }
        }
        fetched = false;
        cp_async_wait_all();                                    // an early fetch of an item without a vector body
        for (long long i = b + tid; i < hb; i += kThreads)
            if (in_bounds(i, 1, b, e, n)) pull16_scalar<T, M>(x, center, w, lambda, oml, i);
        for (long long i = te + tid; i < e; i += kThreads)
            if (in_bounds(i, 1, b, e, n)) pull16_scalar<T, M>(x, center, w, lambda, oml, i);
        item += gridDim.x;
        if (item < item_end) locate(item);
    }
}

// Steps 4-5 on 16-bit parameters for any M and any alignment (scalar).
template <typename T>
__global__ void __launch_bounds__(kThreads)
center_pull16_generic_kernel(MutPtrs x, T* __restrict__ center, const float* __restrict__ beta,
                             const Segment* __restrict__ segs, int per_layer, int item_begin, long long n, int tile,
                             float lambda, int M)
{
    grid_dependency_sync();
    long long b, e;
    const float* __restrict__ bt = beta;
    if (per_layer) {
        const Segment sg = segs[item_begin + blockIdx.x];
        b = sg.begin;
        e = b + sg.len;
        bt = beta + static_cast<size_t>(sg.layer) * M;
    } else {
        b = static_cast<long long>(item_begin + blockIdx.x) * tile;
        e = min(n, b + tile);
    }
    __shared__ float w[kMaxWorkers];
    if (threadIdx.x < M) w[threadIdx.x] = bt[threadIdx.x];
    __syncthreads();
    const float oml = 1.0f - lambda;
    for (long long i = b + threadIdx.x; i < e; i += kThreads) {
        if (!in_bounds(i, 1, b, e, n)) continue;
        float c = w[0] * Pair16<T>::load1(reinterpret_cast<const T*>(x.p[0]) + i);
        for (int m = 1; m < M; ++m) c = fmaf(w[m], Pair16<T>::load1(reinterpret_cast<const T*>(x.p[m]) + i), c);
        if (center) Pair16<T>::store1(center + i, c);
        for (int m = 0; m < M; ++m) {
            T* p = reinterpret_cast<T*>(x.p[m]) + i;
            Pair16<T>::store1(p, fmaf(lambda, c, oml * Pair16<T>::load1(p)));
        }
    }
}

// Proximity step on 16-bit parameters and centre: x_m <- round(fmaf(a, x_C, (1-a) x_m)), fp32 arithmetic on
// the widened values, one rounding per stored value (a = 0 leaves the workers' bits untouched,
// a = 1 makes them bit-equal to the centre).  One CTA per flat tile; the centre column (eight
// elements, 16 bytes) is loaded once and reused for all M workers.
template <typename T>
__global__ void __launch_bounds__(kThreads)
prox16_kernel(MutPtrs x, const T* __restrict__ center, long long n, int tile, float a, int M, int vec_ok)
{
    grid_dependency_sync();
    const long long b = static_cast<long long>(blockIdx.x) * tile;
    const long long e = min(n, b + tile);
    const float oma = 1.0f - a;
    long long hb, te;
    split_range16(b, e, vec_ok, hb, te);
    const int ncol = static_cast<int>((te - hb) >> 3);
    for (int c = threadIdx.x; c < ncol; c += kThreads) {
        if (!in_bounds(hb + 8LL * c, 8, b, e, n)) continue;
        float cc[8];
        unpack8<T>(__ldcs(reinterpret_cast<const uint4*>(center + hb) + c), cc);
        int m = 0;
        for (; m + 4 <= M; m += 4) {
            uint4 raw[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) raw[q] = __ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(x.p[m + q]) + hb) + c);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float v[8];
                unpack8<T>(raw[q], v);
#pragma unroll
                for (int t = 0; t < 8; ++t) v[t] = fmaf(a, cc[t], oma * v[t]);
                __stcs(reinterpret_cast<uint4*>(reinterpret_cast<T*>(x.p[m + q]) + hb) + c, pack8<T>(v));
            }
        }
        for (; m < M; ++m) {
            float v[8];
            unpack8<T>(__ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(x.p[m]) + hb) + c), v);
#pragma unroll
            for (int t = 0; t < 8; ++t) v[t] = fmaf(a, cc[t], oma * v[t]);
            __stcs(reinterpret_cast<uint4*>(reinterpret_cast<T*>(x.p[m]) + hb) + c, pack8<T>(v));
        }
    }
    for (int pass = 0; pass < 2; ++pass) {
        const long long lo = pass ? te : b, hi = pass ? e : hb;
        for (long long i = lo + threadIdx.x; i < hi; i += kThreads) {
            if (!in_bounds(i, 1, b, e, n)) continue;
            const float c = Pair16<T>::load1(center + i);
            for (int m = 0; m < M; ++m) {
                T* p = reinterpret_cast<T*>(x.p[m]) + i;
                Pair16<T>::store1(p, fmaf(a, c, oma * Pair16<T>::load1(p)));
            }
        }
    }
}

// M = 1 on 16-bit parameters: the centre is a copy of the single worker.
template <typename T>
__global__ void __launch_bounds__(kThreads)
copy16_kernel(const T* __restrict__ src, T* __restrict__ dst, long long n)
{
    grid_dependency_sync();
    const long long stride = static_cast<long long>(gridDim.x) * kThreads;
    for (long long i = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x; i < n; i += stride)
        if (in_bounds(i, 1, 0, n, n)) dst[i] = src[i];
}

}  // namespace grawa
