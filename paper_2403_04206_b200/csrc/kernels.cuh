// Device code of libgrawa: segmented sum of squares, score/weight finalisation,
// fused centre + pull, proximity step.  Written for sm_100a; HBM-bandwidth bound,
// plain ALU arithmetic (a small-M weighted sum is not a dense contraction).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace grawa {

constexpr int kMaxWorkers = 64;
constexpr int kThreads = 256;          // threads per CTA of the streaming kernels
constexpr int kFinalizeThreads = 256;
constexpr int kStageDoubles = 1024;    // shared-memory staging of the finalisation (8 KB)
constexpr int kMaxRegWorkers = 16;     // largest M the register-resident centre+pull kernel is built for

enum Variant { kGrawa = 0, kMgrawa = 1, kLgrawa = 2 };
enum StatusBits { kStatusNonFinite = 1, kStatusTimeout = 2 };

struct ConstPtrs { const float* p[kMaxWorkers]; };
struct MutPtrs { float* p[kMaxWorkers]; };

// One work item: elements [begin, begin+len) of the flat vector, all inside layer `layer`.
// Items are cut at layer boundaries and at absolute multiples of the tile size, so every
// interior boundary is 16-byte aligned relative to the base pointer.
struct Segment {
    long long begin;
    int len;
    int layer;
};

// Programmatic dependent launch: every kernel first waits until the grids it depends on have
// completed and their writes are visible, then lets its own dependents start launching.  The
// dependents wait the same way, so only launch latency and CTA ramp-up overlap, never data.
// Both instructions do nothing in a kernel launched without the attribute.
__device__ __forceinline__ void grid_dependency_sync()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Debug build (-DGRAWA_DEBUG_BOUNDS): every global access of the streaming kernels is first checked
// against the vector's length; a violation is counted and the access skipped (nothing traps).
// In the normal build the check is the constant `true` and costs nothing.
#ifdef GRAWA_DEBUG_BOUNDS
__device__ int g_bounds_violations = 0;
__device__ __forceinline__ bool in_bounds(long long first, long long count, long long total)
{
    if (first >= 0 && count >= 0 && first + count <= total) return true;
    atomicAdd(&g_bounds_violations, 1);
    return false;
}
// Arithmetic-only check of the checker itself: three ranges that are out of bounds, one that is not.
__global__ void bounds_selfcheck_kernel()
{
    if (threadIdx.x == 0) {
        (void)in_bounds(-1, 1, 10);
        (void)in_bounds(8, 4, 10);
        (void)in_bounds(10, 1, 10);
        (void)in_bounds(6, 4, 10);
    }
}
#else
__device__ __forceinline__ bool in_bounds(long long, long long, long long) { return true; }
#endif

// Streaming accesses: every byte is touched once per step, so keep it out of the way in L1/L2
// (ld.global.cs / st.global.cs; measured equal to .nc.L1::no_allocate loads and better than
// default-cached loads for the sum of squares).
__device__ __forceinline__ float4 ld_stream4(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ float ld_stream1(const float* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream4(float4* p, float4 v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream1(float* p, float v) { __stcs(p, v); }

// Splits [b, e) into scalar head [b, hb), 16-byte aligned body [hb, te), scalar tail [te, e).
// With vec_ok == 0 (a base pointer that is not 16-byte aligned) everything is head.
__device__ __forceinline__ void split_range(long long b, long long e, int vec_ok, long long& hb, long long& te)
{
    if (vec_ok) {
        hb = min((b + 3) & ~3LL, e);
        te = max(e & ~3LL, hb);
    } else {
        hb = e;
        te = e;
    }
}

// Deterministic block sum of one double per thread: xor-free shuffle-down tree inside each warp,
// then thread 0 adds the warp results in warp order.  Result valid in thread 0.
template <int THREADS>
__device__ __forceinline__ double block_sum_fixed_order(double v)
{
    __shared__ double warp_part[THREADS / 32];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_down_sync(0xffffffffu, v, d);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) warp_part[warp] = v;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < THREADS / 32; ++w) total += warp_part[w];
    }
    return total;
}

// Everything the sum-of-squares and finalisation code needs to know about one step.
struct StepScratch {
    const Segment* segs;           // sum-of-squares work items of one worker, C of them
    const int* layer_seg_first;    // first item of each layer, K+1 entries
    int C, K, M, variant;
    long long n;                   // elements per worker (bounds checks of the debug build)
    double* partials;              // [M][C]
    double* S;                     // [K][M]
    double* A;                     // [K+1][M]: per-layer terms, then the per-worker scores in row K
    float* beta;                   // [K][M] (LGRAWA) or [M]
    int* layer_flag;               // [K] non-finite flag of each layer's group (LGRAWA)
    unsigned* global_ticket;       // zero between steps
    unsigned global_target;        // arrivals that complete the step's finalisation
    int* status;                   // written (not or-ed) when the finalisation completes
    unsigned* work_counter;        // cleared for the bulk-copy centre+pull kernel
    const double* given;           // [given_parts][K][M] given per-layer norms or sums of squares, else NULL
    int given_parts;               // parts (e.g. ranks) whose sums are added in part order; 1 for norms
    int given_sums;                // 1: `given` holds sums of squares, 0: norms
    float* weights_out;            // optional copies
    double* scores_out;
    double* sumsq_out;
};

// Step 3 for one group of M scores (Eq. 2 / 4 / 7) with the zero-score limit and the non-finite
// fallback, computed by the whole CTA: thread m < M passes its score `a` and gets beta_m back.
// The reciprocals are taken in parallel and added by one thread in worker order, so the value is
// the one a sequential loop over m = 0..M-1 gives.  Every thread of the CTA must call it.
struct WeightsSmem {
    double r[kMaxWorkers];
    double z;
};

__device__ __forceinline__ float weights_parallel(double a, int M, WeightsSmem& sm, int& flagged)
{
    const int tid = threadIdx.x;
    const bool active = tid < M;
    const bool fin = active && isfinite(a);
    const bool zero = fin && a == 0.0;
    const int finite = __syncthreads_count(fin);
    const int zeros = __syncthreads_count(zero);
    if (active) sm.r[tid] = (fin && !zero) ? 1.0 / a : 0.0;
    __syncthreads();
    if (tid == 0) {
        double z = 0.0;
        for (int m = 0; m < M; ++m) z += sm.r[m];     // adding the 0.0 of a skipped worker is exact
        sm.z = z;
    }
    __syncthreads();
    flagged = finite < M;
    double w = 0.0;
    if (active) {
        if (finite == 0) w = 1.0 / M;
        else if (zeros > 0) w = zero ? 1.0 / zeros : 0.0;
        else w = fin ? sm.r[tid] / sm.z : 0.0;
    }
    return static_cast<float>(w);
}

struct FinalizeSmem {
    double layer_sum[kMaxWorkers];
    WeightsSmem w;
    double stage[kStageDoubles];
    int flag;
};

// Steps 1b-3 for one non-empty layer, by a whole CTA of kThreads threads.  Warp w adds the partials
// of workers w, w+8, ... of layer k in a fixed order into S[k][m]; the layer's terms sqrt(S) (S
// itself for the flat norm) go to row k of A; LGRAWA turns them into the layer's weights (Eq. 7).
// With `given` set no partials are read: either the given norm of (layer, worker) takes the place
// of sqrt(S) (the running estimates of the Local variants), or S is the sum, in part order, of
// given partial sums of squares (element-range shards of the vector on several GPUs).
__device__ __forceinline__ void finalize_layer(const StepScratch& sc, int k, FinalizeSmem& sm)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int M = sc.M;
    if (sc.given == nullptr) {
        const int s0 = sc.layer_seg_first[k], s1 = sc.layer_seg_first[k + 1];
        for (int m = warp; m < M; m += kThreads / 32) {
            const double* row = sc.partials + static_cast<size_t>(m) * sc.C;
            // eight independent running sums per lane keep eight loads in flight; the order in which
            // they are combined is fixed, so the sum is the same on every run
            double part[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
            int s = s0 + lane;
            for (; s + 7 * 32 < s1; s += 8 * 32) {
#pragma unroll
                for (int u = 0; u < 8; ++u) part[u] += __ldcg(row + s + u * 32);
            }
            for (int u = 0; s < s1; s += 32, ++u) part[u] += __ldcg(row + s);
            double acc = ((part[0] + part[1]) + (part[2] + part[3])) + ((part[4] + part[5]) + (part[6] + part[7]));
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, d);
            if (lane == 0) sm.layer_sum[m] = acc;
        }
    }
    __syncthreads();
    double term = 0.0;
    const size_t idx = static_cast<size_t>(k) * M + tid;
    if (tid < M) {
        double s;
        if (sc.given == nullptr) {
            s = sm.layer_sum[tid];
            term = (sc.variant == kGrawa) ? s : sqrt(s);
        } else if (sc.given_sums) {                // sums of squares of the parts, added in part order
            s = 0.0;
            for (int r = 0; r < sc.given_parts; ++r) s += sc.given[static_cast<size_t>(r) * sc.K * M + idx];
            term = (sc.variant == kGrawa) ? s : sqrt(s);
        } else {                                   // the caller's norm estimate stands in for sqrt(S)
            const double a = sc.given[idx];
            s = a * a;
            term = (sc.variant == kGrawa) ? s : a;
        }
        sc.S[idx] = s;
        if (sc.sumsq_out) sc.sumsq_out[idx] = s;
        sc.A[idx] = term;
    }
    if (sc.variant == kLgrawa) {
        int flagged = 0;
        const float w = weights_parallel(term, M, sm.w, flagged);
        if (tid < M) {
            if (sc.scores_out) sc.scores_out[idx] = term;
            sc.beta[idx] = w;
            if (sc.weights_out) sc.weights_out[idx] = w;
        }
        if (tid == 0) sc.layer_flag[k] = flagged;
    }
}

// Called by a whole CTA after its part of the finalisation.  The CTA that makes the count reach
// `global_target` finishes the step: rows of empty layers, MGRAWA / GRAWA scores (the K rows of A
// added per worker in layer order, Eq. 3 / Eq. 2) and weights (Eq. 4), the status word, and the
// reset of the counters for the next step.  No CTA waits for another.
__device__ __forceinline__ void finalize_arrive(const StepScratch& sc, FinalizeSmem& sm)
{
    const int tid = threadIdx.x;
    const int M = sc.M, K = sc.K;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const bool last = atomicAdd(sc.global_ticket, 1u) == sc.global_target - 1u;
        if (last) *sc.global_ticket = 0u;
        sm.flag = last;
    }
    __syncthreads();
    if (!sm.flag) return;
    __threadfence();

    // empty layers: zero sums and terms, uniform weights (they are never applied).  With given
    // norms or sums every layer has been processed, whether it has local elements or not.
    const bool all_layers = sc.given != nullptr;
    for (int k = tid; k < K; k += kThreads) {
        if (all_layers || sc.layer_seg_first[k] != sc.layer_seg_first[k + 1]) continue;
        for (int m = 0; m < M; ++m) {
            const size_t idx = static_cast<size_t>(k) * M + m;
            sc.S[idx] = 0.0;
            sc.A[idx] = 0.0;
            if (sc.sumsq_out) sc.sumsq_out[idx] = 0.0;
            if (sc.variant == kLgrawa) {
                const float u = static_cast<float>(1.0 / M);
                sc.beta[idx] = u;
                if (sc.weights_out) sc.weights_out[idx] = u;
                if (sc.scores_out) sc.scores_out[idx] = 0.0;
            }
        }
    }
    int flagged = 0;
    if (sc.variant == kLgrawa) {
        int f = 0;
        for (int k = tid; k < K; k += kThreads)
            if (all_layers || sc.layer_seg_first[k] != sc.layer_seg_first[k + 1]) f |= __ldcg(sc.layer_flag + k);
        flagged = __syncthreads_or(f);
    } else {
        // Rows of A are staged through shared memory in blocks (parallel loads); thread m then adds
        // its column in layer order.  Rows of empty layers count as 0.
        const int rows_per_block = kStageDoubles / M;
        double a = 0.0;
        for (int k0 = 0; k0 < K; k0 += rows_per_block) {
            const int rows = min(rows_per_block, K - k0);
            for (int i = tid; i < rows * M; i += kThreads) {
                const int k = k0 + i / M;
                const bool empty = !all_layers && sc.layer_seg_first[k] == sc.layer_seg_first[k + 1];
                sm.stage[i] = empty ? 0.0 : __ldcg(sc.A + static_cast<size_t>(k0) * M + i);
            }
            __syncthreads();
            if (tid < M)
                for (int r = 0; r < rows; ++r) a += sm.stage[r * M + tid];
            __syncthreads();
        }
        if (tid < M) {
            if (sc.variant == kGrawa) a = sqrt(a);
            sc.A[static_cast<size_t>(K) * M + tid] = a;
            if (sc.scores_out) sc.scores_out[tid] = a;
        }
        const float w = weights_parallel(a, M, sm.w, flagged);
        if (tid < M) {
            sc.beta[tid] = w;
            if (sc.weights_out) sc.weights_out[tid] = w;
        }
    }
    if (tid == 0) {
        *sc.status = flagged ? kStatusNonFinite : 0;
        *sc.work_counter = 0u;
    }
}

// ---------------------------------------------------------------------------------------------
// Step 1 (Eq. 3 / Eq. 5): partial[m][s] = sum of g_m[j]^2 over segment s.  Work items are the
// (worker, segment) pairs, worker-major; CTA b takes items b, b + gridDim.x, ...  fp32 squares
// are accumulated in runs of UNROLL terms per accumulator and the runs are combined in fp64; the
// order depends only on the item, never on the grid, so results are reproducible.
// ---------------------------------------------------------------------------------------------
// Six CTAs per SM (at most 42 registers): measured 1.4x faster than four on the large workloads.
template <int UNROLL>
__global__ void __launch_bounds__(kThreads, 6)
sumsq_kernel(ConstPtrs grads, StepScratch sc, int items, int vec_ok)
{
    grid_dependency_sync();
    __shared__ double warp_part[2][kThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int C = sc.C;

    int parity = 0;
    for (int item = blockIdx.x; item < items; item += gridDim.x, parity ^= 1) {
        const int m = item / C;
        const int s = item - m * C;
        const Segment sg = sc.segs[s];
        const float* __restrict__ g = grads.p[m];
        const long long b = sg.begin, e = b + sg.len;
        long long hb, te;
        split_range(b, e, vec_ok, hb, te);
        double dacc = 0.0;

        const float4* __restrict__ g4 = reinterpret_cast<const float4*>(g + hb);
        const int ncol = static_cast<int>((te - hb) >> 2);
        for (int c0 = 0; c0 < ncol; c0 += kThreads * UNROLL) {
            float4 v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int c = c0 + u * kThreads + tid;
                v[u] = (c < ncol && in_bounds(hb + 4LL * c, 4, sc.n)) ? ld_stream4(g4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                a0 = fmaf(v[u].x, v[u].x, a0);
                a1 = fmaf(v[u].y, v[u].y, a1);
                a2 = fmaf(v[u].z, v[u].z, a2);
                a3 = fmaf(v[u].w, v[u].w, a3);
            }
            dacc += (static_cast<double>(a0) + static_cast<double>(a1)) +
                    (static_cast<double>(a2) + static_cast<double>(a3));
        }
        for (long long i = b + tid; i < hb; i += kThreads) {
            const double v = in_bounds(i, 1, sc.n) ? static_cast<double>(ld_stream1(g + i)) : 0.0;
            dacc += v * v;
        }
        for (long long i = te + tid; i < e; i += kThreads) {
            const double v = in_bounds(i, 1, sc.n) ? static_cast<double>(ld_stream1(g + i)) : 0.0;
            dacc += v * v;
        }
        // Fixed-order block sum.  Two alternating buffers need only one barrier per item: a warp
        // can write buffer p again only after the barrier of the item in between, which thread 0
        // reaches after it has read buffer p.
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) dacc += __shfl_down_sync(0xffffffffu, dacc, d);
        if (lane == 0) warp_part[parity][warp] = dacc;
        __syncthreads();
        if (tid == 0) {
            double total = 0.0;
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) total += warp_part[parity][w];
            sc.partials[static_cast<size_t>(m) * C + s] = total;
        }
    }
}

// Steps 1b-3: one CTA per layer reduces the layer's partials and, for LGRAWA, computes its
// weights; the CTA that arrives last completes the step (see finalize_arrive).
// (Folding this into the sum-of-squares kernel with one ticket per layer was measured slower: the
// fence and atomic each CTA then needs before it can retire cost more than the launch they save.)
__global__ void __launch_bounds__(kThreads)
finalize_kernel(StepScratch sc)
{
    grid_dependency_sync();
    __shared__ FinalizeSmem fsm;
    const int k = blockIdx.x;
    if (sc.given != nullptr || sc.layer_seg_first[k] != sc.layer_seg_first[k + 1]) finalize_layer(sc, k, fsm);
    finalize_arrive(sc, fsm);
}

// ---------------------------------------------------------------------------------------------
// Steps 4-5, register variant: one thread owns a 16-byte column of all M workers, so each
// parameter is read once and M independent vector loads are in flight per column.
//   x_C = sum_m beta_m x_m   (fp32 FMA chain, m = 0..M-1)      x_m <- fmaf(pull, x_C, (1-pull) x_m)
// PER_LAYER: the items are the Segments, weights of the segment's layer (Eq. 7); otherwise flat
// tiles of `tile` elements and one weight per worker (Eq. 2 / Eq. 4).  The launch covers items
// [item_begin, item_end); CTA b takes items item_begin + b, + gridDim.x, ...
// ---------------------------------------------------------------------------------------------
template <int M>
__device__ __forceinline__ void pull_scalar(const MutPtrs& x, float* center, const float (&w)[M],
                                            float lambda, float oml, long long i)
{
    float v[M];
#pragma unroll
    for (int m = 0; m < M; ++m) v[m] = ld_stream1(x.p[m] + i);
    float c = w[0] * v[0];
#pragma unroll
    for (int m = 1; m < M; ++m) c = fmaf(w[m], v[m], c);
    if (center) st_stream1(center + i, c);
#pragma unroll
    for (int m = 0; m < M; ++m) st_stream1(x.p[m] + i, fmaf(lambda, c, oml * v[m]));
}

// Shape of the register kernel for M workers: a thread keeps COLS columns of VEC floats of all M
// workers in flight (COLS * M vector loads) and a CTA covers kThreads * COLS * VEC elements per
// pass.  Measured alternatives: 8-byte columns with more CTAs per SM lose badly at M = 16 and
// change nothing for M <= 8 (the kernel sits at the mixed read/write rate of the memory system).
__host__ __device__ constexpr int pull_cols(int M) { return (M <= 2) ? 8 : (M <= 4) ? 4 : (M <= 8) ? 2 : 1; }
__host__ __device__ constexpr int pull_vec(int) { return 4; }
__host__ __device__ constexpr int pull_pass_elems(int M) { return kThreads * pull_cols(M) * pull_vec(M); }

template <int VEC> struct VecIO;
template <> struct VecIO<4> {
    static __device__ __forceinline__ void ld(const float* p, float (&o)[4]) { const float4 t = __ldcs(reinterpret_cast<const float4*>(p)); o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w; }
    static __device__ __forceinline__ void st(float* p, const float (&o)[4]) { __stcs(reinterpret_cast<float4*>(p), make_float4(o[0], o[1], o[2], o[3])); }
};
template <> struct VecIO<2> {
    static __device__ __forceinline__ void ld(const float* p, float (&o)[2]) { const float2 t = __ldcs(reinterpret_cast<const float2*>(p)); o[0] = t.x; o[1] = t.y; }
    static __device__ __forceinline__ void st(float* p, const float (&o)[2]) { __stcs(reinterpret_cast<float2*>(p), make_float2(o[0], o[1])); }
};

template <int M, bool PER_LAYER>
__global__ void __launch_bounds__(kThreads, 2)
center_pull_kernel(MutPtrs x, float* __restrict__ center, const float* __restrict__ beta,
                   const Segment* __restrict__ segs, int item_begin, int item_end, long long n, int tile, float lambda,
                   int vec_ok)
{
    grid_dependency_sync();
    constexpr int COLS = pull_cols(M);
    constexpr int VEC = pull_vec(M);
    const float oml = 1.0f - lambda;
    const int tid = threadIdx.x;
    float w[M];
    if (!PER_LAYER) {
#pragma unroll
        for (int m = 0; m < M; ++m) w[m] = beta[m];
    }
    for (int item = item_begin + blockIdx.x; item < item_end; item += gridDim.x) {
        long long b, e;
        if (PER_LAYER) {
            const Segment sg = segs[item];
            b = sg.begin;
            e = b + sg.len;
            const float* __restrict__ bt = beta + static_cast<size_t>(sg.layer) * M;
#pragma unroll
            for (int m = 0; m < M; ++m) w[m] = bt[m];
        } else {
            b = static_cast<long long>(item) * tile;
            e = min(n, b + tile);
        }
        long long hb, te;
        split_range(b, e, vec_ok, hb, te);
        const int ncol = static_cast<int>((te - hb) / VEC);      // te - hb is a multiple of 4
        for (int c0 = 0; c0 < ncol; c0 += kThreads * COLS) {
            float v[COLS][M][VEC];
#pragma unroll
            for (int q = 0; q < COLS; ++q) {
                const int c = c0 + q * kThreads + tid;
                if (c < ncol && in_bounds(hb + static_cast<long long>(c) * VEC, VEC, n)) {
#pragma unroll
                    for (int m = 0; m < M; ++m) VecIO<VEC>::ld(x.p[m] + hb + static_cast<long long>(c) * VEC, v[q][m]);
                }
            }
#pragma unroll
            for (int q = 0; q < COLS; ++q) {
                const int c = c0 + q * kThreads + tid;
                if (c < ncol && in_bounds(hb + static_cast<long long>(c) * VEC, VEC, n)) {
                    float cc[VEC];
#pragma unroll
                    for (int t = 0; t < VEC; ++t) cc[t] = w[0] * v[q][0][t];
#pragma unroll
                    for (int m = 1; m < M; ++m) {
#pragma unroll
                        for (int t = 0; t < VEC; ++t) cc[t] = fmaf(w[m], v[q][m][t], cc[t]);
                    }
                    if (center) VecIO<VEC>::st(center + hb + static_cast<long long>(c) * VEC, cc);
#pragma unroll
                    for (int m = 0; m < M; ++m) {
                        float o[VEC];
#pragma unroll
                        for (int t = 0; t < VEC; ++t) o[t] = fmaf(lambda, cc[t], oml * v[q][m][t]);
                        VecIO<VEC>::st(x.p[m] + hb + static_cast<long long>(c) * VEC, o);
                    }
                }
            }
        }
        for (long long i = b + tid; i < hb; i += kThreads)
            if (in_bounds(i, 1, n)) pull_scalar<M>(x, center, w, lambda, oml, i);
        for (long long i = te + tid; i < e; i += kThreads)
            if (in_bounds(i, 1, n)) pull_scalar<M>(x, center, w, lambda, oml, i);
    }
}

// Steps 4-5 for any M up to kMaxWorkers and any alignment: scalar, two passes over the workers
// (the second pass re-reads the elements the same thread has just read, from cache).
__global__ void __launch_bounds__(kThreads)
center_pull_generic_kernel(MutPtrs x, float* __restrict__ center, const float* __restrict__ beta,
                           const Segment* __restrict__ segs, int per_layer, int item_begin, long long n,
                           int tile, float lambda, int M)
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
        if (!in_bounds(i, 1, n)) continue;
        float c = w[0] * x.p[0][i];
        for (int m = 1; m < M; ++m) c = fmaf(w[m], x.p[m][i], c);
        if (center) center[i] = c;
        for (int m = 0; m < M; ++m) x.p[m][i] = fmaf(lambda, c, oml * x.p[m][i]);
    }
}

// Running gradient-norm estimate of the Local variants (appendix algorithm, taken literally):
// g_mvg <- gamma g_mvg + (1-gamma) g_cur ; g_est <- gamma g_mvg / corr, corr = 1 - gamma^t.
__global__ void __launch_bounds__(kThreads)
norm_ema_kernel(double* __restrict__ g_mvg, const double* __restrict__ g_cur, int K, double gamma, double corr,
                double* __restrict__ g_est)
{
    grid_dependency_sync();
    const int k = blockIdx.x * kThreads + threadIdx.x;
    if (k < K) {
        const double v = gamma * g_mvg[k] + (1.0 - gamma) * g_cur[k];
        g_mvg[k] = v;
        g_est[k] = gamma * v / corr;
    }
}

// M = 1: the centre is the single worker; the worker itself is left untouched.
__global__ void __launch_bounds__(kThreads)
copy_kernel(const float* __restrict__ src, float* __restrict__ dst, long long n, int vec_ok)
{
    grid_dependency_sync();
    const long long stride = static_cast<long long>(gridDim.x) * kThreads;
    const long long t = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x;
    const long long n4 = vec_ok ? (n >> 2) : 0;
    for (long long c = t; c < n4; c += stride)
        st_stream4(reinterpret_cast<float4*>(dst) + c, ld_stream4(reinterpret_cast<const float4*>(src) + c));
    for (long long i = (n4 << 2) + t; i < n; i += stride) dst[i] = src[i];
}

// Proximity step (the "Prox." update of Algorithms 1-2): x_m <- fmaf(a, x_C, (1-a) x_m), a = mu/tau.
// One CTA per flat tile; the centre column is loaded once and reused for all M workers.
__global__ void __launch_bounds__(kThreads)
prox_kernel(MutPtrs x, const float* __restrict__ center, long long n, int tile, float a, int M, int vec_ok)
{
    grid_dependency_sync();
    const long long b = static_cast<long long>(blockIdx.x) * tile;
    const long long e = min(n, b + tile);
    const float oma = 1.0f - a;
    long long hb, te;
    split_range(b, e, vec_ok, hb, te);
    const int ncol = static_cast<int>((te - hb) >> 2);
    for (int c = threadIdx.x; c < ncol; c += kThreads) {
        if (!in_bounds(hb + 4LL * c, 4, n)) continue;
        const float4 cc = ld_stream4(reinterpret_cast<const float4*>(center + hb) + c);
        int m = 0;
        for (; m + 4 <= M; m += 4) {
            float4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] = ld_stream4(reinterpret_cast<const float4*>(x.p[m + q] + hb) + c);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float4 o;
                o.x = fmaf(a, cc.x, oma * v[q].x); o.y = fmaf(a, cc.y, oma * v[q].y);
                o.z = fmaf(a, cc.z, oma * v[q].z); o.w = fmaf(a, cc.w, oma * v[q].w);
                st_stream4(reinterpret_cast<float4*>(x.p[m + q] + hb) + c, o);
            }
        }
        for (; m < M; ++m) {
            const float4 v = ld_stream4(reinterpret_cast<const float4*>(x.p[m] + hb) + c);
            float4 o;
            o.x = fmaf(a, cc.x, oma * v.x); o.y = fmaf(a, cc.y, oma * v.y);
            o.z = fmaf(a, cc.z, oma * v.z); o.w = fmaf(a, cc.w, oma * v.w);
            st_stream4(reinterpret_cast<float4*>(x.p[m] + hb) + c, o);
        }
    }
    for (int pass = 0; pass < 2; ++pass) {
        const long long lo = pass ? te : b, hi = pass ? e : hb;
        for (long long i = lo + threadIdx.x; i < hi; i += kThreads) {
            if (!in_bounds(i, 1, n)) continue;
            const float c = center[i];
            for (int m = 0; m < M; ++m) x.p[m][i] = fmaf(a, c, oma * x.p[m][i]);
        }
    }
}

}  // namespace grawa
