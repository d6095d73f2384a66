// Centre + pull (Eq. 4 / Eq. 7 and the distributed update of Algorithms 1-2) for more workers than
// the register kernels cover: the worker count is a run-time value and the columns wait in shared
// memory.  One kernel for fp32, bfloat16 and half storage.
#pragma once
#include "kernels.cuh"
#include "kernels_16bit.cuh"

namespace grawa {

// Column type of the any-M staged kernel: ELEMS elements in 16 bytes, widened to / rounded from fp32.
template <typename T> struct Column16B {
    static constexpr int ELEMS = 8;
    static __device__ __forceinline__ void widen(const uint4& r, float (&v)[8]) { unpack8<T>(r, v); }
    static __device__ __forceinline__ uint4 narrow(const float (&v)[8]) { return pack8<T>(v); }
    static __device__ __forceinline__ float load1(const T* p) { return Pair16<T>::load1(p); }
    static __device__ __forceinline__ void store1(T* p, float v) { Pair16<T>::store1(p, v); }
};
template <> struct Column16B<float> {
    static constexpr int ELEMS = 4;
    static __device__ __forceinline__ void widen(const uint4& r, float (&v)[4])
    {
        v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y); v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
    }
    static __device__ __forceinline__ uint4 narrow(const float (&v)[4])
    {
        return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
    }
    static __device__ __forceinline__ float load1(const float* p) { return *p; }
    static __device__ __forceinline__ void store1(float* p, float v) { *p = v; }
};

// CTA size of the any-M staged kernel: the largest multiple of 32 threads (at most 256) whose M
// 16-byte slots per thread stay within 72 KB of shared memory, so that three CTAs fit on an SM.
__host__ __device__ constexpr int staged_any_threads(int M)
{
    const int fit = (72 * 1024 / 16) / M / 32 * 32;
    return fit > 256 ? 256 : (fit < 32 ? 32 : fit);
}

// Steps 4-5 for 17..64 workers (any storage type): the staging of center_pull16_staged_kernel with the
// worker count a run-time value: every thread copies its 16-byte column of each worker to its own
// slots of shared memory with `cp.async`, waits for its own copies, and walks the workers twice
// from shared memory (centre: fp32 FMA chain over m = 0..M-1; pull; one rounding per stored value).
// Shared memory: M x blockDim.x x 16 bytes for the columns plus M weights.
template <typename T, bool PER_LAYER>
__global__ void __launch_bounds__(256, 3)
center_pull_staged_any_kernel(const __grid_constant__ MutPtrs x, T* __restrict__ center, const float* __restrict__ beta, const Segment* __restrict__ segs,
                              int item_begin, int item_end, long long n, int tile, float lambda, int M, int preload)
{
    constexpr int E = Column16B<T>::ELEMS;
    extern __shared__ __align__(16) uint4 stage_any[];        // [M][blockDim.x] columns, then M weights
    const int tid = threadIdx.x, threads = blockDim.x;
    float* w = reinterpret_cast<float*>(stage_any + static_cast<size_t>(M) * threads);
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
        hb = min((b + E - 1) / E * E, e);                       // 16-byte aligned body, scalar head and tail
        te = max(e / E * E, hb);
        ncol = static_cast<int>((te - hb) / E);
    };
    auto fetch = [&](int c) {
        if (c < ncol && in_bounds(hb + static_cast<long long>(E) * c, E, b, e, n)) {
            for (int m = 0; m < M; ++m)
                cp_async16(&stage_any[m * threads + tid], reinterpret_cast<const T*>(x.p[m]) + hb + static_cast<long long>(E) * c);
        }
    };
    auto edge = [&](long long i) {                               // one unaligned edge element, straight in global memory
        float c = w[0] * Column16B<T>::load1(reinterpret_cast<const T*>(x.p[0]) + i);
        for (int m = 1; m < M; ++m) c = fmaf(w[m], Column16B<T>::load1(reinterpret_cast<const T*>(x.p[m]) + i), c);
        if (center) Column16B<T>::store1(center + i, c);
        for (int m = 0; m < M; ++m) {
            T* p = reinterpret_cast<T*>(x.p[m]) + i;
            Column16B<T>::store1(p, fmaf(lambda, c, (1.0f - lambda) * Column16B<T>::load1(p)));
        }
    };
    bool fetched = false;
    if (item < item_end) {
        locate(item);
        if (preload) {                                          // see center_pull_kernel for when this is valid
            fetch(tid);
            fetched = true;
        }
    }
    grid_dependency_sync();
    const float oml = 1.0f - lambda;
    while (item < item_end) {
        __syncthreads();                                        // nobody still reads the previous item's weights
        for (int m = tid; m < M; m += threads) w[m] = PER_LAYER ? beta[static_cast<size_t>(layer) * M + m] : beta[m];
        __syncthreads();
        for (int c = tid; c < ncol; c += threads) {
            if (!fetched) fetch(c);
            fetched = false;
            cp_async_wait_all();
            if (!in_bounds(hb + static_cast<long long>(E) * c, E, b, e, n)) continue;
            const uint4* col = stage_any + tid;
            float cc[E];
            {
                float v[E];
                Column16B<T>::widen(col[0], v);
#pragma unroll
                for (int t = 0; t < E; ++t) cc[t] = w[0] * v[t];
            }
#pragma unroll 4
            for (int m = 1; m < M; ++m) {
                float v[E];
                Column16B<T>::widen(col[m * threads], v);
#pragma unroll
                for (int t = 0; t < E; ++t) cc[t] = fmaf(w[m], v[t], cc[t]);
            }
            if (center) __stcs(reinterpret_cast<uint4*>(center + hb) + c, Column16B<T>::narrow(cc));
#pragma unroll 4
            for (int m = 0; m < M; ++m) {
                float v[E];
                Column16B<T>::widen(col[m * threads], v);
#pragma unroll
                for (int t = 0; t < E; ++t) v[t] = fmaf(lambda, cc[t], oml * v[t]);
                __stcs(reinterpret_cast<uint4*>(reinterpret_cast<T*>(x.p[m]) + hb) + c, Column16B<T>::narrow(v));
            }
        }
        fetched = false;
        cp_async_wait_all();                                    // an early fetch of an item without a vector body
        for (long long i = b + tid; i < hb; i += threads)
            if (in_bounds(i, 1, b, e, n)) edge(i);
        for (long long i = te + tid; i < e; i += threads)
            if (in_bounds(i, 1, b, e, n)) edge(i);
        item += gridDim.x;
        if (item < item_end) locate(item);
    }
}

}  // namespace grawa
