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

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Trace build (-DGRAWA_TRACE): the three kernels of a step stamp the device's nanosecond timer when
// their first CTA enters, when the first and the last CTA get past the dependency wait, and when
// the last CTA leaves, one row per launch (see grawa_trace_read).  Nothing is skipped or reordered;
// thread 0 of every CTA issues one counting atomic and four min/max reductions.  In the normal
// build the tracer is an empty object.
#ifdef GRAWA_TRACE
struct TraceRow { unsigned long long first_entry, first_go, last_go, last_exit; };
constexpr int kTraceKinds = 3;         // 0 sum of squares, 1 finalisation, 2 centre+pull
constexpr int kTraceRows = 64;         // launches of one kind wrap around after this many
__device__ TraceRow g_trace[kTraceRows][kTraceKinds];
__device__ unsigned g_trace_arrivals[kTraceKinds];
struct KernelTrace {
    unsigned long long t_entry = 0, t_go = 0;
    unsigned arrival = 0;
    int kind;
    __device__ __forceinline__ explicit KernelTrace(int k) : kind(k)
    {
        if (threadIdx.x == 0) {
            t_entry = global_timer_ns();
            arrival = atomicAdd(&g_trace_arrivals[kind], 1u);
        }
    }
    __device__ __forceinline__ void go() { if (threadIdx.x == 0) t_go = global_timer_ns(); }
    __device__ __forceinline__ void done()
    {
        if (threadIdx.x != 0) return;
        TraceRow& r = g_trace[(arrival / gridDim.x) % kTraceRows][kind];
        atomicMin(&r.first_entry, t_entry);
        atomicMin(&r.first_go, t_go);
        atomicMax(&r.last_go, t_go);
        atomicMax(&r.last_exit, global_timer_ns());
    }
};
#else
struct KernelTrace {
    __device__ __forceinline__ explicit KernelTrace(int) {}
    __device__ __forceinline__ void go() {}
    __device__ __forceinline__ void done() {}
};
#endif

// Debug build (-DGRAWA_DEBUG_BOUNDS): every global access of the streaming kernels is first checked
// against the work item it belongs to, [lo, hi), which itself must lie inside the vector [0, total);
// every index into scratch memory is checked against the size of its table.  A violation is counted
// and the access skipped (nothing traps).  In the normal build the checks are the constant `true`
// and cost nothing.
#ifdef GRAWA_DEBUG_BOUNDS
__device__ int g_bounds_violations = 0;
__device__ __forceinline__ bool in_bounds(long long first, long long count, long long lo, long long hi, long long total)
{
    if (count >= 0 && lo >= 0 && hi <= total && first >= lo && first + count <= hi) return true;
    atomicAdd(&g_bounds_violations, 1);
    return false;
}
__device__ __forceinline__ bool scratch_ok(long long index, long long limit)
{
    if (index >= 0 && index < limit) return true;
    atomicAdd(&g_bounds_violations, 1);
    return false;
}
// Arithmetic-only check of the checker itself: six triples that must be counted (outside the vector,
// inside the vector but outside the item, an item that sticks out of the vector, a scratch index at
// its limit), two that must not.
__global__ void bounds_selfcheck_kernel()
{
    if (threadIdx.x == 0) {
        (void)in_bounds(-1, 1, 0, 10, 10);
        (void)in_bounds(8, 4, 0, 10, 10);
        (void)in_bounds(10, 1, 0, 10, 10);
        (void)in_bounds(6, 4, 0, 8, 10);        // in the vector, past the end of the item
        (void)in_bounds(2, 1, 3, 8, 10);        // in the vector, in front of the item
        (void)in_bounds(6, 2, 4, 12, 10);       // the item itself leaves the vector
        (void)scratch_ok(5, 5);
        (void)in_bounds(6, 4, 4, 10, 10);
        (void)scratch_ok(4, 5);
    }
}
#else
__device__ __forceinline__ bool in_bounds(long long, long long, long long, long long, long long) { return true; }
__device__ __forceinline__ bool scratch_ok(long long, long long) { return true; }
#endif

// Streaming accesses: every byte is touched once per step, so keep it out of the way in L1/L2
// (ld.global.cs / st.global.cs; measured equal to .nc.L1::no_allocate loads and better than
// default-cached loads for the sum of squares).
__device__ __forceinline__ float4 ld_stream4(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ float ld_stream1(const float* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream4(float4* p, float4 v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream1(float* p, float v) { __stcs(p, v); }

// Hint: bring `bytes` (a multiple of 16) from the 16-byte aligned address p into L2.  No architectural
// effect; L2 is the GPU's point of coherence, so a prefetched line can never be stale.
__device__ __forceinline__ void prefetch_l2(const void* p, unsigned bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

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

// ---------------------------------------------------------------------------------------------
// Exact accumulation of the sums of squares.  S[k][m] of one step is kept as a fixed-point integer
// of kBinWords 32-bit digits, each digit in its own 64-bit word (32 bits of head-room for carries, so
// a word absorbs 2^32 additions before it could overflow), least significant bit 2^-149, the
// smallest positive fp32 value.  A CTA adds its fp64 partial sum with up to three integer atomic
// adds that return nothing.  Integer addition is associative: the total does not depend on the
// order in which the CTAs arrive, so the result is bitwise reproducible without a second reduction
// pass over stored partial sums.  Digits below 2^-149 (they can only come from the fp64 squares of
// a layer's few unaligned edge elements) are dropped; a partial sum that is not finite or is
// >= 2^170 sets the row's marker word instead and the row reads back as +infinity.
// ---------------------------------------------------------------------------------------------
constexpr int kBinWords = 10;          // digits: bit positions 0..319, values below 2^171
constexpr int kRowWords = 11;          // words per (layer, worker) row: the digits and the marker
constexpr int kBinLsbExp = -149;
constexpr int kBinMaxExp = 170;        // partial sums must be < 2^170

// Layout: digit-major, [copy][kRowWords][K][M] words, so that the threads of a warp that read the same
// digit of neighbouring (layer, worker) rows touch neighbouring words.  `row` points at digit 0 of
// a (layer, worker) pair and `stride` = K * M is the distance between its digits.
__device__ __forceinline__ void bins_add(unsigned long long* __restrict__ row, size_t stride, double v)
{
    if (!(v < 1.4965776766268446e51)) {                 // 2^170; also catches NaN
        atomicOr(row + kBinWords * stride, 1ull);
        return;
    }
    const unsigned long long bits = static_cast<unsigned long long>(__double_as_longlong(v));
    const int ex = static_cast<int>((bits >> 52) & 0x7ffu);
    if (ex == 0) return;                                // zero, or an fp64 subnormal (far below 2^-149)
    unsigned long long man = (bits & 0x000fffffffffffffull) | 0x0010000000000000ull;    // v = man * 2^(ex - 1075)
    int sh = ex - 1075 - kBinLsbExp;                    // bit position of man's least significant bit
    if (sh < 0) {
        if (sh <= -53) return;
        man >>= -sh;
        sh = 0;
    }
    const int b0 = sh >> 5, r = sh & 31;
    const unsigned long long lo = man << r;             // bits 0..63 of man * 2^r
    const unsigned long long hi = r ? (man >> (64 - r)) : 0ull;    // bits 64..84
    const unsigned long long d0 = lo & 0xffffffffull, d1 = lo >> 32;
    if (!scratch_ok(b0 + (hi ? 2 : d1 ? 1 : 0), kBinWords)) return;       // debug build: the digits stay inside the row
    if (d0) atomicAdd(row + b0 * stride, d0);
    if (d1) atomicAdd(row + (b0 + 1) * stride, d1);
    if (hi) atomicAdd(row + (b0 + 2) * stride, hi);     // b0 + 2 <= 9 because v < 2^170
}

// The value of a row: digits added from the most significant one down (a fixed order).  The digit
// rows exist twice (see StepScratch) and the copy not in use is all zeros, so the reader adds the
// two copies digit by digit instead of first finding out which one holds the sums: all loads are
// independent of one another.
__device__ __forceinline__ double bins_value(const unsigned long long* __restrict__ row, size_t stride)
{
    const size_t copy_words = stride * kRowWords;
    unsigned long long w[kBinWords + 1];
#pragma unroll
    for (int b = 0; b <= kBinWords; ++b) w[b] = __ldcg(row + b * stride) + __ldcg(row + copy_words + b * stride);
    if (w[kBinWords]) return __longlong_as_double(0x7ff0000000000000ll);      // +infinity
    double s = 0.0;
#pragma unroll
    for (int b = kBinWords - 1; b >= 0; --b) {
        const double scale = __longlong_as_double(static_cast<long long>(1023 + 32 * b + kBinLsbExp) << 52);   // 2^(32 b - 149)
        s += static_cast<double>(w[b]) * scale;
    }
    return s;
}

// Everything the sum-of-squares and finalisation code needs to know about one step.
//
// The digit rows exist twice.  A sum-of-squares kernel adds into the copy named by *next_buf and
// clears the other copy for the step after it; the finalisation that consumes the sums (it adds the
// two copies, one of which is zero) then points the word at the other copy.  The word is written
// only while none of its readers can be running (the kernels of a step follow one another on the
// stream), and it lives in device memory, so a replayed CUDA graph alternates between the copies
// like eager calls do.
struct StepScratch {
    const Segment* segs;           // sum-of-squares work items of one worker, C of them
    int C, K, M, variant;
    long long n;                   // elements per worker (bounds checks of the debug build)
    int prefetch_stride, prefetch_waves;   // sum-of-squares kernel: L2 prefetch of later items by the first CTAs (0 = none)
    unsigned long long* bins;      // [2][kRowWords][K][M]
    int* next_buf;                 // copy the next sum-of-squares kernel adds into
    double* S;                     // [K][M]
    double* A;                     // [K+1][M]: per-layer terms, then the per-worker scores in row K
    float* beta;                   // [K][M] (LGRAWA) or [M]
    int* status;                   // rewritten by every finalisation
    int* status_copy;              // optional caller-owned copy of the status word, else NULL
    unsigned* work_counter;        // cleared for the bulk-copy centre+pull kernel
    const double* given;           // [given_parts][K][M] given per-layer norms or sums of squares, else NULL
    int given_parts;               // parts (e.g. ranks) whose sums are added in part order; 1 for norms
    int given_sums;                // 1: `given` holds sums of squares, 0: norms
    float* weights_out;            // optional copies
    double* scores_out;
    double* sumsq_out;
};

__device__ __forceinline__ size_t bins_copy_words(const StepScratch& sc) { return static_cast<size_t>(sc.K) * sc.M * kRowWords; }

// End of a sum-of-squares CTA's work: clear this CTA's share of the other copy of the digit rows.
__device__ __forceinline__ void bins_turnover(const StepScratch& sc, int buf)
{
    const size_t words = bins_copy_words(sc);
    unsigned long long* other = sc.bins + static_cast<size_t>(buf ^ 1) * words;
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < words; i += static_cast<size_t>(gridDim.x) * blockDim.x)
        other[i] = 0ull;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *sc.status = 0;                  // the finalisation that follows only adds flags to it
        if (sc.status_copy) *sc.status_copy = 0;
    }
}

// Step 3 for one group of M <= 64 scores (Eq. 2 / 4 / 7) with the zero-score limit and the
// non-finite fallback, by one full warp: lane l passes the scores of workers l and l + 32 and gets
// their weights back.  The reciprocals are taken in parallel and added in worker order by every
// lane (shuffles), so the normaliser is the value a sequential loop over m = 0..M-1 gives.
__device__ __forceinline__ void weights_warp(double a0, double a1, int M, float& w0, float& w1, int& flagged)
{
    const int lane = threadIdx.x & 31;
    const bool act0 = lane < M, act1 = lane + 32 < M;
    const bool fin0 = act0 && isfinite(a0), fin1 = act1 && isfinite(a1);
    const bool zero0 = fin0 && a0 == 0.0, zero1 = fin1 && a1 == 0.0;
    const int finite = __popc(__ballot_sync(0xffffffffu, fin0)) + __popc(__ballot_sync(0xffffffffu, fin1));
    const int zeros = __popc(__ballot_sync(0xffffffffu, zero0)) + __popc(__ballot_sync(0xffffffffu, zero1));
    const double r0 = (fin0 && !zero0) ? 1.0 / a0 : 0.0;      // adding the 0.0 of a skipped worker is exact
    const double r1 = (fin1 && !zero1) ? 1.0 / a1 : 0.0;
    double z = 0.0;
    for (int m = 0; m < M && m < 32; ++m) z += __shfl_sync(0xffffffffu, r0, m);
    for (int m = 32; m < M; ++m) z += __shfl_sync(0xffffffffu, r1, m - 32);
    flagged = finite < M;
    double v0 = 0.0, v1 = 0.0;
    if (finite == 0) {
        v0 = act0 ? 1.0 / M : 0.0;
        v1 = act1 ? 1.0 / M : 0.0;
    } else if (zeros > 0) {
        v0 = zero0 ? 1.0 / zeros : 0.0;
        v1 = zero1 ? 1.0 / zeros : 0.0;
    } else {
        v0 = fin0 ? r0 / z : 0.0;
        v1 = fin1 ? r1 / z : 0.0;
    }
    w0 = static_cast<float>(v0);
    w1 = static_cast<float>(v1);
}

// S[k][m] of one row from whichever source the step has: the digit rows of the sum-of-squares
// kernel, given partial sums of squares added in part order (element-range shards on several GPUs),
// or a given norm estimate (the running estimates of the Local variants).
__device__ __forceinline__ double row_sumsq(const StepScratch& sc, const unsigned long long* __restrict__ bins, size_t idx)
{
    if (sc.given == nullptr) return bins_value(bins + idx, static_cast<size_t>(sc.K) * sc.M);
    if (sc.given_sums) {
        double s = 0.0;
        const size_t stride = static_cast<size_t>(sc.K) * sc.M;
#pragma unroll 4
        for (int p = 0; p < sc.given_parts; ++p) s += __ldcg(sc.given + p * stride + idx);
        return s;
    }
    const double a = __ldcg(sc.given + idx);
    return a * a;
}

// The row's term: its norm (the given estimate itself where there is one), or S for the flat norm.
__device__ __forceinline__ double row_term(const StepScratch& sc, size_t idx, double s)
{
    if (sc.variant == kGrawa) return s;
    if (sc.given != nullptr && !sc.given_sums) return __ldcg(sc.given + idx);
    return sqrt(s);
}

__device__ __forceinline__ void store_row(const StepScratch& sc, size_t idx, double s, double term)
{
    if (!scratch_ok(static_cast<long long>(idx), static_cast<long long>(sc.K) * sc.M)) return;
    sc.S[idx] = s;
    sc.A[idx] = term;
    if (sc.sumsq_out) sc.sumsq_out[idx] = s;
}

// ---------------------------------------------------------------------------------------------
// Steps 2-3: S -> scores -> weights.
// LGRAWA: one warp per layer, any number of CTAs, no CTA depends on another (Eq. 5-7).
// MGRAWA / GRAWA: one CTA; thread (p, m) adds worker m's terms of a contiguous run of layers (one
// layer when the CTA has a thread per row) in layer order, the runs are added in run order in two
// levels (Eq. 3 / Eq. 2), one warp normalises (Eq. 4).
// Every sum has a fixed order.  The status word is rewritten by every launch.
// ---------------------------------------------------------------------------------------------
constexpr int kFinThreadsLayered = 256;     // LGRAWA: 8 layers per CTA
constexpr int kFinThreadsFlat = 1024;       // MGRAWA / GRAWA: the one CTA (at most)
constexpr int kFinGroupSlots = 512;         // >= ceil(sqrt(P)) * M for every P * M <= 1024, M <= 64
constexpr int kFinSharedOutRows = 4096;     // MGRAWA / GRAWA with more (layer, worker) rows than this: several CTAs
constexpr int kFinGivenLayersOneCta = 256;  // LGRAWA from given scores with more layers than this: several CTAs
constexpr int kFinTicketWord = 3;           // word of the scratch's leading block that counts those CTAs' tickets

__global__ void __launch_bounds__(kFinThreadsFlat, 1)
finalize_kernel(StepScratch sc)
{
    __shared__ double part_sm[kFinThreadsFlat];
    __shared__ double group_sm[kFinGroupSlots];
    __shared__ double score_sm[kMaxWorkers];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int M = sc.M, K = sc.K;
    KernelTrace trace(1);
    grid_dependency_sync();
    trace.go();

    const unsigned long long* bins = sc.bins;
    // the first thread turns the copies of the digit rows over; the load is issued now, the store
    // at the very end, so that nothing waits for it
    const bool keeper = blockIdx.x == 0 && tid == 0;
    int next = 0;
    if (keeper) {
        *sc.work_counter = 0u;
        if (sc.given == nullptr) next = __ldcg(sc.next_buf) ^ 1;
    }

    if (sc.variant == kLgrawa) {
        int any_flag = 0;
        const int warps = blockDim.x >> 5;
        for (int k = blockIdx.x * warps + warp; k < K; k += gridDim.x * warps) {
            const size_t base = static_cast<size_t>(k) * M;
            double a0 = 0.0, a1 = 0.0;
            if (lane < M) {
                const double s = row_sumsq(sc, bins, base + lane);
                a0 = row_term(sc, base + lane, s);
                store_row(sc, base + lane, s, a0);
            }
            if (lane + 32 < M) {
                const double s = row_sumsq(sc, bins, base + lane + 32);
                a1 = row_term(sc, base + lane + 32, s);
                store_row(sc, base + lane + 32, s, a1);
            }
            float w0, w1;
            int flagged;
            weights_warp(a0, a1, M, w0, w1, flagged);
            any_flag |= flagged;
            if (lane < M) {
                sc.beta[base + lane] = w0;
                if (sc.weights_out) sc.weights_out[base + lane] = w0;
                if (sc.scores_out) sc.scores_out[base + lane] = a0;
            }
            if (lane + 32 < M) {
                sc.beta[base + lane + 32] = w1;
                if (sc.weights_out) sc.weights_out[base + lane + 32] = w1;
                if (sc.scores_out) sc.scores_out[base + lane + 32] = a1;
            }
        }
        // the status word: a launch of one CTA (always the case with given scores, where no
        // sum-of-squares kernel has cleared the word) writes it; several CTAs only add their flags
        const int cta_flag = __syncthreads_or(any_flag);
        if (tid == 0) {
            if (gridDim.x == 1) {
                *sc.status = cta_flag ? kStatusNonFinite : 0;
                if (sc.status_copy) *sc.status_copy = cta_flag ? kStatusNonFinite : 0;
            } else if (cta_flag) {
                atomicOr(sc.status, kStatusNonFinite);
                if (sc.status_copy) atomicOr(sc.status_copy, kStatusNonFinite);
            }
        }
        if (keeper && sc.given == nullptr) *sc.next_buf = next;
        trace.done();
        return;
    }

    // MGRAWA / GRAWA: one CTA, or (many rows) several CTAs that share the rows out and a last one to
    // finish, whichever it is, that adds the stored terms in the same fixed order as the one CTA would
    const int P = max(1, min(K, static_cast<int>(blockDim.x) / M));
    const int run = (K + P - 1) / P;
    const bool shared_out = gridDim.x > 1;
    if (shared_out) {
        const long long rows = static_cast<long long>(K) * M;
        for (long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + tid; idx < rows;
             idx += static_cast<long long>(gridDim.x) * blockDim.x) {
            const double s = row_sumsq(sc, bins, static_cast<size_t>(idx));
            store_row(sc, static_cast<size_t>(idx), s, row_term(sc, static_cast<size_t>(idx), s));
        }
        // one ticket per CTA (no CTA waits for another): the rows are fenced before the ticket is
        // taken, and whoever takes the last one reads all of them behind a fence of its own
        unsigned* ticket = reinterpret_cast<unsigned*>(sc.next_buf) + kFinTicketWord;
        __shared__ int last_sm;
        __threadfence();
        __syncthreads();
        if (tid == 0) last_sm = atomicAdd(ticket, 1u) == gridDim.x - 1 ? 1 : 0;
        __syncthreads();
        if (!last_sm) {
            if (keeper && sc.given == nullptr) *sc.next_buf = next;
            trace.done();
            return;
        }
        __threadfence();
        if (tid == 0) *ticket = 0u;                              // ready for the next launch
    }
    if (tid < P * M) {
        const int p = tid / M, m = tid - p * M;
        const int k1 = min(K, (p + 1) * run);
        double a = 0.0;
        if (shared_out) {                                        // the stored terms, same order; loads eight at a time
            int k = p * run;
            for (; k + 8 <= k1; k += 8) {
                double t[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) t[u] = __ldcg(sc.A + static_cast<size_t>(k + u) * M + m);
#pragma unroll
                for (int u = 0; u < 8; ++u) a += t[u];
            }
            for (; k < k1; ++k) a += __ldcg(sc.A + static_cast<size_t>(k) * M + m);
        } else {
            for (int k = p * run; k < k1; ++k) {
                const size_t idx = static_cast<size_t>(k) * M + m;
                const double s = row_sumsq(sc, bins, idx);
                const double term = row_term(sc, idx, s);
                store_row(sc, idx, s, term);
                a += term;
            }
        }
        part_sm[tid] = a;
    }
    __syncthreads();
    // the P runs of a worker are added in two levels, both in run order: G groups of L consecutive runs
    int G = 1;
    while (G * G < P) ++G;
    const int L = (P + G - 1) / G;
    if (tid < G * M) {
        const int j = tid / M, m = tid - j * M;
        const int p1 = min(P, (j + 1) * L);
        double a = 0.0;
        for (int p = j * L; p < p1; ++p) a += part_sm[p * M + m];
        group_sm[tid] = a;
    }
    __syncthreads();
    if (tid < M) {
        double a = 0.0;
        for (int j = 0; j < G; ++j) a += group_sm[j * M + tid];
        if (sc.variant == kGrawa) a = sqrt(a);
        sc.A[static_cast<size_t>(K) * M + tid] = a;
        if (sc.scores_out) sc.scores_out[tid] = a;
        score_sm[tid] = a;
    }
    __syncthreads();
    if (warp == 0) {
        const double a0 = lane < M ? score_sm[lane] : 0.0;
        const double a1 = lane + 32 < M ? score_sm[lane + 32] : 0.0;
        float w0, w1;
        int flagged;
        weights_warp(a0, a1, M, w0, w1, flagged);
        if (lane < M) {
            sc.beta[lane] = w0;
            if (sc.weights_out) sc.weights_out[lane] = w0;
        }
        if (lane + 32 < M) {
            sc.beta[lane + 32] = w1;
            if (sc.weights_out) sc.weights_out[lane + 32] = w1;
        }
        if (lane == 0) {
            *sc.status = flagged ? kStatusNonFinite : 0;
            if (sc.status_copy) *sc.status_copy = flagged ? kStatusNonFinite : 0;
        }
    }
    if (keeper && sc.given == nullptr) *sc.next_buf = next;
    trace.done();
}

// ---------------------------------------------------------------------------------------------
// Step 1 (Eq. 3 / Eq. 5): S[k][m] += sum of g_m[j]^2 over segment s of layer k.  Work items are the
// (worker, segment) pairs, worker-major; CTA b takes items b, b + gridDim.x, ...  fp32 squares
// are accumulated in runs of UNROLL terms per accumulator, the runs are combined in fp64 in an order
// that depends only on the item, and the item's sum is added exactly (integer digits) to its row:
// the result does not depend on the grid or on the order in which items finish.
// ---------------------------------------------------------------------------------------------
// Six CTAs per SM (at most 42 registers): measured 1.4x faster than four on the large workloads.
template <int UNROLL>
__global__ void __launch_bounds__(kThreads, 6)
sumsq_kernel(const __grid_constant__ ConstPtrs grads, StepScratch sc, int items, int vec_ok)
{
    __shared__ double warp_part[2][kThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int C = sc.C;
    // the work list belongs to the plan, not to the kernel before this one: fetch the first item early
    Segment first_sg = Segment{0, 0, 0};
    if (static_cast<int>(blockIdx.x) < items) first_sg = sc.segs[blockIdx.x % C];
    // On short problems the CTAs that are resident when the kernel starts ask for the gradients of
    // the items one, two, ... grid-fuls further on to be brought into L2 while they wait for the
    // kernel in front (whose tail leaves DRAM partly idle).  Hints only; see prefetch_l2.
    if (static_cast<int>(blockIdx.x) < sc.prefetch_stride && tid < sc.prefetch_waves) {
        const long long it = blockIdx.x + static_cast<long long>(tid + 1) * sc.prefetch_stride;
        if (it < items) {
            const int pm = static_cast<int>(it / C);
            const Segment sg = sc.segs[it - static_cast<long long>(pm) * C];
            long long phb, pte;
            split_range(sg.begin, sg.begin + sg.len, vec_ok, phb, pte);
            const unsigned bytes = static_cast<unsigned>(pte - phb) * 4u;
            if (bytes > 0 && in_bounds(phb, pte - phb, sg.begin, sg.begin + sg.len, sc.n)) prefetch_l2(grads.p[pm] + phb, bytes);
        }
    }
    KernelTrace trace(0);
    grid_dependency_sync();
    trace.go();
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
                v[u] = (c < ncol && in_bounds(hb + 4LL * c, 4, b, e, sc.n)) ? ld_stream4(g4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
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
            const double v = in_bounds(i, 1, b, e, sc.n) ? static_cast<double>(ld_stream1(g + i)) : 0.0;
            dacc += v * v;
        }
        for (long long i = te + tid; i < e; i += kThreads) {
            const double v = in_bounds(i, 1, b, e, sc.n) ? static_cast<double>(ld_stream1(g + i)) : 0.0;
            dacc += v * v;
        }
        // Fixed-order block sum.  Two alternating buffers need only one barrier per item: a warp
        // can write buffer p again only after the barrier of the item in between, which thread 0
        // reaches after it has read buffer p.
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
    trace.done();
}

// ---------------------------------------------------------------------------------------------
// Steps 4-5, register variant: one thread owns a 16-byte (VEC = 4) or 32-byte (VEC = 8) column of
// all M workers, so each parameter is read once and M independent vector loads are in flight per column.
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
//
// VEC = 8 (32-byte loads and stores, `ld/st.global.v8.f32`) keeps the same bytes per thread in half
// as many columns and needs 32-byte aligned bases; an arithmetic-free copy of this access shape runs
// 1.2-1.4 % faster with 32-byte than with 16-byte accesses at M = 4, 8 and 16.  Above 8 workers
// a 32-byte column of all workers takes about 210 registers, so those CTAs have 128 threads (two per
// SM, the same bytes in flight).  A pass covers the same number of elements for either width.
__host__ __device__ constexpr int pull_cols(int M, int VEC = 4)
{
    return VEC == 8 ? ((M <= 2) ? 4 : (M <= 4) ? 2 : 1) : ((M <= 2) ? 8 : (M <= 4) ? 4 : (M <= 8) ? 2 : 1);
}
__host__ __device__ constexpr int pull_threads(int M, int VEC = 4) { return (VEC == 8 && M > 8) ? kThreads / 2 : kThreads; }
__host__ __device__ constexpr int pull_pass_elems(int M) { return kThreads * pull_cols(M) * 4; }
static_assert(pull_threads(16, 8) * pull_cols(16, 8) * 8 == pull_pass_elems(16) && pull_threads(8, 8) * pull_cols(8, 8) * 8 == pull_pass_elems(8) &&
              pull_threads(4, 8) * pull_cols(4, 8) * 8 == pull_pass_elems(4) && pull_threads(2, 8) * pull_cols(2, 8) * 8 == pull_pass_elems(2),
              "a pass covers the same elements for both access widths");

// [b, e) split into scalar head, body aligned to VEC elements, scalar tail (everything head without vec_ok).
template <int VEC>
__device__ __forceinline__ void split_range_vec(long long b, long long e, int vec_ok, long long& hb, long long& te)
{
    if (vec_ok) {
        hb = min((b + (VEC - 1)) & ~static_cast<long long>(VEC - 1), e);
        te = max(e & ~static_cast<long long>(VEC - 1), hb);
    } else {
        hb = e;
        te = e;
    }
}

template <int VEC> struct VecIO;
template <> struct VecIO<4> {
    static __device__ __forceinline__ void ld(const float* p, float (&o)[4]) { const float4 t = __ldcs(reinterpret_cast<const float4*>(p)); o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w; }
    static __device__ __forceinline__ void st(float* p, const float (&o)[4]) { __stcs(reinterpret_cast<float4*>(p), make_float4(o[0], o[1], o[2], o[3])); }
};
template <> struct VecIO<8> {
    static __device__ __forceinline__ void ld(const float* p, float (&o)[8])
    {
        asm volatile("ld.global.cs.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(o[0]), "=f"(o[1]), "=f"(o[2]), "=f"(o[3]), "=f"(o[4]), "=f"(o[5]), "=f"(o[6]), "=f"(o[7]) : "l"(p) : "memory");
    }
    static __device__ __forceinline__ void st(float* p, const float (&o)[8])
    {
        asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     :: "l"(p), "f"(o[0]), "f"(o[1]), "f"(o[2]), "f"(o[3]), "f"(o[4]), "f"(o[5]), "f"(o[6]), "f"(o[7]) : "memory");
    }
};
template <> struct VecIO<2> {
    static __device__ __forceinline__ void ld(const float* p, float (&o)[2]) { const float2 t = __ldcs(reinterpret_cast<const float2*>(p)); o[0] = t.x; o[1] = t.y; }
    static __device__ __forceinline__ void st(float* p, const float (&o)[2]) { __stcs(reinterpret_cast<float2*>(p), make_float2(o[0], o[1])); }
};

// `preload` != 0: the first chunk of parameters is loaded BEFORE the dependency wait, so that these
// loads overlap the tail of the kernels that produce the weights.  Only valid when every kernel
// that may still be running at that point leaves the parameters alone, i.e. when the kernels in
// front of this one on the stream are this library's own sum-of-squares / finalisation kernels
// (they pass their own dependency wait before they let this kernel start, so whatever the caller
// ran earlier has completed by then).
//
// With `prefetch_waves` > 0 the first `prefetch_stride` CTAs (the ones resident when the kernel
// starts) also ask, before the wait, for the parameters of the items `prefetch_stride`,
// 2 * `prefetch_stride`, ... further on to be brought into L2: while the weights are being finalised
// DRAM has nothing else to do, and the CTAs that take those items later find them in L2.  A
// prefetch is a hint without architectural effect, and L2 is the GPU's point of coherence.
template <int M, bool PER_LAYER, int VEC>
__global__ void __launch_bounds__(pull_threads(M, VEC), 2)
center_pull_kernel(MutPtrs x, float* __restrict__ center, const float* __restrict__ beta,
                   const Segment* __restrict__ segs, int item_begin, int item_end, long long n, int tile, float lambda,
                   int vec_ok, int preload, int prefetch_stride, int prefetch_waves)
{
    constexpr int COLS = pull_cols(M, VEC);
    constexpr int THREADS = pull_threads(M, VEC);
    const int tid = threadIdx.x;
    int item = item_begin + blockIdx.x;
    // the work list belongs to the plan, not to the kernel before this one: fetch the first item early
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
        split_range_vec<VEC>(b, e, vec_ok, hb, te);
        ncol = static_cast<int>((te - hb) / VEC);               // te - hb is a multiple of VEC
    };
    float v[COLS][M][VEC];
    auto load_chunk = [&](int c0) {
#pragma unroll
        for (int q = 0; q < COLS; ++q) {
            const int c = c0 + q * THREADS + tid;
            if (c < ncol && in_bounds(hb + static_cast<long long>(c) * VEC, VEC, b, e, n)) {
#pragma unroll
                for (int m = 0; m < M; ++m) VecIO<VEC>::ld(x.p[m] + hb + static_cast<long long>(c) * VEC, v[q][m]);
            }
        }
    };
    bool loaded = false;
    if (item < item_end) {
        locate(item);
        if (preload) {
            // (not compiled in for M > 8, where the kernel has no registers to spare and problems are large)
            if (M <= 8 && static_cast<int>(blockIdx.x) < prefetch_stride && tid < M * prefetch_waves) {
                const int m = tid % M;
                const long long it = item + static_cast<long long>(tid / M + 1) * prefetch_stride;
                if (it < item_end) {
                    long long pb, pe, phb, pte;
                    if (PER_LAYER) {
                        const Segment sg = segs[it];
                        pb = sg.begin;
                        pe = pb + sg.len;
                    } else {
                        pb = it * tile;
                        pe = min(n, pb + tile);
                    }
                    split_range_vec<VEC>(pb, pe, vec_ok, phb, pte);
                    const unsigned bytes = static_cast<unsigned>(pte - phb) * 4u;       // a multiple of 16
                    const float* base = x.p[0];
#pragma unroll
                    for (int mm = 1; mm < M; ++mm)
                        if (mm == m) base = x.p[mm];                // a select chain: no run-time index into the pointer table
                    if (bytes > 0 && in_bounds(phb, pte - phb, pb, pe, n)) prefetch_l2(base + phb, bytes);
                }
            }
            load_chunk(0);
            loaded = true;
        }
    }
    KernelTrace trace(2);
    grid_dependency_sync();
    trace.go();
    const float oml = 1.0f - lambda;
    float w[M];
    if (!PER_LAYER) {
#pragma unroll
        for (int m = 0; m < M; ++m) w[m] = beta[m];
    }
    while (item < item_end) {
        if (PER_LAYER) {
            const float* __restrict__ bt = beta + static_cast<size_t>(layer) * M;
#pragma unroll
            for (int m = 0; m < M; ++m) w[m] = bt[m];
        }
        for (int c0 = 0; c0 < ncol; c0 += THREADS * COLS) {
            if (!loaded) load_chunk(c0);
            loaded = false;
#pragma unroll
            for (int q = 0; q < COLS; ++q) {
                const int c = c0 + q * THREADS + tid;
                if (c < ncol && in_bounds(hb + static_cast<long long>(c) * VEC, VEC, b, e, n)) {
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
        loaded = false;                                  // an item without a vector body used nothing
        for (long long i = b + tid; i < hb; i += THREADS)
            if (in_bounds(i, 1, b, e, n)) pull_scalar<M>(x, center, w, lambda, oml, i);
        for (long long i = te + tid; i < e; i += THREADS)
            if (in_bounds(i, 1, b, e, n)) pull_scalar<M>(x, center, w, lambda, oml, i);
        item += gridDim.x;
        if (item < item_end) locate(item);
    }
    trace.done();
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
        if (!in_bounds(i, 1, b, e, n)) continue;
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
        if (in_bounds(4 * c, 4, 0, n, n)) st_stream4(reinterpret_cast<float4*>(dst) + c, ld_stream4(reinterpret_cast<const float4*>(src) + c));
    for (long long i = (n4 << 2) + t; i < n; i += stride)
        if (in_bounds(i, 1, 0, n, n)) dst[i] = src[i];
}

// Proximity step (the "Prox." update of Algorithms 1-2): x_m <- fmaf(a, x_C, (1-a) x_m), a = mu/tau.
// One CTA per flat tile; the centre column is loaded once and reused for all M workers.  VEC = 4
// (16-byte columns) or 8 (32-byte columns, bases 32-byte aligned).
template <int VEC>
__global__ void __launch_bounds__(kThreads)
prox_kernel(MutPtrs x, const float* __restrict__ center, long long n, int tile, float a, int M, int vec_ok)
{
    grid_dependency_sync();
    const long long b = static_cast<long long>(blockIdx.x) * tile;
    const long long e = min(n, b + tile);
    const float oma = 1.0f - a;
    long long hb, te;
    split_range_vec<VEC>(b, e, vec_ok, hb, te);
    const int ncol = static_cast<int>((te - hb) / VEC);
    for (int c = threadIdx.x; c < ncol; c += kThreads) {
        const long long j = hb + static_cast<long long>(VEC) * c;
        if (!in_bounds(j, VEC, b, e, n)) continue;
        float cc[VEC];
        VecIO<VEC>::ld(center + j, cc);
        int m = 0;
        for (; m + 4 <= M; m += 4) {
            float v[4][VEC];
#pragma unroll
            for (int q = 0; q < 4; ++q) VecIO<VEC>::ld(x.p[m + q] + j, v[q]);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
#pragma unroll
                for (int t = 0; t < VEC; ++t) v[q][t] = fmaf(a, cc[t], oma * v[q][t]);
                VecIO<VEC>::st(x.p[m + q] + j, v[q]);
            }
        }
        for (; m < M; ++m) {
            float v[VEC];
            VecIO<VEC>::ld(x.p[m] + j, v);
#pragma unroll
            for (int t = 0; t < VEC; ++t) v[t] = fmaf(a, cc[t], oma * v[t]);
            VecIO<VEC>::st(x.p[m] + j, v);
        }
    }
    for (int pass = 0; pass < 2; ++pass) {
        const long long lo = pass ? te : b, hi = pass ? e : hb;
        for (long long i = lo + threadIdx.x; i < hi; i += kThreads) {
            if (!in_bounds(i, 1, b, e, n)) continue;
            const float c = center[i];
            for (int m = 0; m < M; ++m) x.p[m][i] = fmaf(a, c, oma * x.p[m][i]);
        }
    }
}

}  // namespace grawa
