// Steps 4-5, bulk-copy variant: the M slices of a tile are staged through shared memory by 1-D
// bulk asynchronous copies (cp.async.bulk, completion on an mbarrier; no cluster multicast), the
// centre and the pulled workers are computed in place in shared memory and written back by bulk
// stores.  One CTA per SM keeps a ring of stages in flight; work items are claimed from an atomic
// counter so that faster SMs take more of them.
//
// Every wait is bounded: when a barrier does not complete within the time limit the CTA records
// kStatusTimeout in the status word, drains what it has in flight (again bounded) and returns.
#pragma once
#include "kernels.cuh"

namespace grawa {

constexpr int kBulkMaxStages = 8;
constexpr unsigned long long kBulkWaitLimitNs = 2000000000ull;   // a wait gives up after 2 s of wall time

struct BulkStageInfo {
    long long begin;   // first element of the item
    int len;           // elements of the item; -1 = no more work
    int layer;
};

__device__ __forceinline__ unsigned smem_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait; false when `limit_ns` of wall time passed without the phase completing.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long* bar, unsigned parity,
                                                  unsigned long long limit_ns = kBulkWaitLimitNs)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > limit_ns) return false;
    }
}
// global -> shared (this CTA's own shared memory), completion counted in bytes on `bar`.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes, unsigned long long* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// shared -> global, tracked by the issuing thread's bulk async-group.
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, unsigned bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all_but_latest() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Scalar update of one element straight in global memory (unaligned layer edges), any M.
__device__ __forceinline__ void bulk_edge_element(const MutPtrs& x, float* center, const float* __restrict__ bt, int M,
                                                  float lambda, float oml, long long i)
{
    float c = bt[0] * x.p[0][i];
    for (int m = 1; m < M; ++m) c = fmaf(bt[m], x.p[m][i], c);
    if (center) center[i] = c;
    for (int m = 0; m < M; ++m) x.p[m][i] = fmaf(lambda, c, oml * x.p[m][i]);
}

// MT = M (2..16): the column of M values is held in registers.  MT = 0: any M, two passes over
// shared memory.  Shared memory: `stages` stages of (M+1) slices of `tile` floats (slice M is
// the centre).  Launch with kThreads threads and one CTA per SM.
template <int MT, bool PER_LAYER>
__global__ void __launch_bounds__(kThreads, 1)
center_pull_bulk_kernel(MutPtrs x, float* __restrict__ center, const float* __restrict__ beta,
                        const Segment* __restrict__ segs, int item_begin, int item_end, long long n, int tile, int stages,
                        int M_rt,
                        float lambda, unsigned* __restrict__ work_counter, int* __restrict__ status)
{
    grid_dependency_sync();
    extern __shared__ __align__(128) float stage_mem[];
    __shared__ __align__(8) unsigned long long full_bar[kBulkMaxStages];
    __shared__ BulkStageInfo info[kBulkMaxStages];

    const int M = (MT > 0) ? MT : M_rt;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float oml = 1.0f - lambda;
    const size_t slice_floats = static_cast<size_t>(tile);
    const size_t stage_floats = slice_floats * (M + 1);

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) mbar_init(&full_bar[s], 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // Lane 0 of warp 0 keeps one claimed item ahead: the atomic and the Segment read of the item
    // after next are issued when a stage is filled and are only needed at the following fill, so
    // their latency is off the critical path.
    long long nxt_begin = 0;
    int nxt_len = -1, nxt_layer = 0;
    auto claim_next = [&]() {
        nxt_begin = 0; nxt_len = -1; nxt_layer = 0;
        const unsigned item = static_cast<unsigned>(item_begin) + atomicAdd(work_counter, 1u);
        if (item < static_cast<unsigned>(item_end)) {
            if (PER_LAYER) {
                const Segment sg = segs[item];
                nxt_begin = sg.begin; nxt_len = sg.len; nxt_layer = sg.layer;
            } else {
                nxt_begin = static_cast<long long>(item) * tile;
                nxt_len = static_cast<int>(min(static_cast<long long>(tile), n - nxt_begin));
            }
        }
    };
    // Warp 0, all lanes: publish the claimed item in info[s], start its loads into stage s, claim the next.
    auto fill_stage = [&](int s) {
        long long b = nxt_begin;
        int len = nxt_len;
        if (lane == 0) { info[s].begin = b; info[s].len = len; info[s].layer = nxt_layer; }
        b = __shfl_sync(0xffffffffu, b, 0);
        len = __shfl_sync(0xffffffffu, len, 0);
        unsigned bytes = 0;
        long long hb = 0;
        if (len > 0) {
            long long te;
            split_range(b, b + len, 1, hb, te);
            bytes = static_cast<unsigned>(te - hb) * 4u;
        }
        if (bytes > 0 && !in_bounds(hb, bytes / 4, b, b + len, n)) bytes = 0;      // debug build: never copy outside the vector
        if (lane == 0) mbar_arrive_expect_tx(&full_bar[s], bytes * static_cast<unsigned>(M));
        __syncwarp();
        if (bytes > 0) {
            float* dst = stage_mem + static_cast<size_t>(s) * stage_floats;
            for (int m = lane; m < M; m += 32) bulk_load(dst + m * slice_floats, x.p[m] + hb, bytes, &full_bar[s]);
        }
        if (lane == 0) claim_next();
    };

    if (warp == 0 && lane == 0) claim_next();
    if (warp == 0)
        for (int s = 0; s < stages - 1; ++s) fill_stage(s);

    int it = 0;
    bool timed_out = false;
    for (;; ++it) {
        const int s = it % stages;
        const unsigned parity = static_cast<unsigned>(it / stages) & 1u;
        const bool ok = mbar_wait_bounded(&full_bar[s], parity);
        const BulkStageInfo si = info[s];
        float* st = stage_mem + static_cast<size_t>(s) * stage_floats;
        long long hb = 0, te = 0;
        if (ok && si.len > 0) {
            const long long b = si.begin, e = b + si.len;
            split_range(b, e, 1, hb, te);
            const int ncol = static_cast<int>((te - hb) >> 2);
            const float* __restrict__ bt = PER_LAYER ? beta + static_cast<size_t>(si.layer) * M : beta;
            float4* cen = reinterpret_cast<float4*>(st + M * slice_floats);
            if constexpr (MT > 0) {
                float w[MT];
#pragma unroll
                for (int m = 0; m < MT; ++m) w[m] = bt[m];
                for (int c = tid; c < ncol; c += kThreads) {
                    float4 v[MT];
#pragma unroll
                    for (int m = 0; m < MT; ++m) v[m] = reinterpret_cast<const float4*>(st + m * slice_floats)[c];
                    float4 cc;
                    cc.x = w[0] * v[0].x; cc.y = w[0] * v[0].y; cc.z = w[0] * v[0].z; cc.w = w[0] * v[0].w;
#pragma unroll
                    for (int m = 1; m < MT; ++m) {
                        cc.x = fmaf(w[m], v[m].x, cc.x); cc.y = fmaf(w[m], v[m].y, cc.y);
                        cc.z = fmaf(w[m], v[m].z, cc.z); cc.w = fmaf(w[m], v[m].w, cc.w);
                    }
                    cen[c] = cc;
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        float4 o;
                        o.x = fmaf(lambda, cc.x, oml * v[m].x); o.y = fmaf(lambda, cc.y, oml * v[m].y);
                        o.z = fmaf(lambda, cc.z, oml * v[m].z); o.w = fmaf(lambda, cc.w, oml * v[m].w);
                        reinterpret_cast<float4*>(st + m * slice_floats)[c] = o;
                    }
                }
            } else {
                for (int c = tid; c < ncol; c += kThreads) {
                    float4 v = reinterpret_cast<const float4*>(st)[c];
                    float w = bt[0];
                    float4 cc;
                    cc.x = w * v.x; cc.y = w * v.y; cc.z = w * v.z; cc.w = w * v.w;
                    for (int m = 1; m < M; ++m) {
                        v = reinterpret_cast<const float4*>(st + m * slice_floats)[c];
                        w = bt[m];
                        cc.x = fmaf(w, v.x, cc.x); cc.y = fmaf(w, v.y, cc.y);
                        cc.z = fmaf(w, v.z, cc.z); cc.w = fmaf(w, v.w, cc.w);
                    }
                    cen[c] = cc;
                    for (int m = 0; m < M; ++m) {
                        float4* p = reinterpret_cast<float4*>(st + m * slice_floats) + c;
                        v = *p;
                        float4 o;
                        o.x = fmaf(lambda, cc.x, oml * v.x); o.y = fmaf(lambda, cc.y, oml * v.y);
                        o.z = fmaf(lambda, cc.z, oml * v.z); o.w = fmaf(lambda, cc.w, oml * v.w);
                        *p = o;
                    }
                }
            }
            // unaligned layer edges: at most 3 elements on each side, straight in global memory
            for (long long i = b + tid; i < hb; i += kThreads)
                if (in_bounds(i, 1, b, e, n)) bulk_edge_element(x, center, bt, M, lambda, oml, i);
            for (long long i = te + tid; i < e; i += kThreads)
                if (in_bounds(i, 1, b, e, n)) bulk_edge_element(x, center, bt, M, lambda, oml, i);
        }
        fence_async_proxy();                          // this thread's shared-memory writes -> async proxy
        if (__syncthreads_or(ok ? 0 : 1)) { timed_out = true; break; }   // uniform: some thread's wait ran out
        if (info[s].len < 0) break;                   // uniform: the work list is exhausted

        if (warp == 0) {
            const unsigned bytes = static_cast<unsigned>(te - hb) * 4u;
            if (bytes > 0 && in_bounds(hb, bytes / 4, si.begin, si.begin + si.len, n)) {
                for (int m = lane; m < M; m += 32) bulk_store(x.p[m] + hb, st + m * slice_floats, bytes);
                if (lane == 0 && center) bulk_store(center + hb, st + M * slice_floats, bytes);
            }
            bulk_commit();
            // The stage consumed one iteration ago is free once its stores have read shared memory.
            bulk_wait_read_all_but_latest();
            __syncwarp();
            fill_stage((it + stages - 1) % stages);
        }
    }

    if (warp == 0) bulk_wait_all();
    if (timed_out) {
        if (tid == 0) atomicOr(status, kStatusTimeout);
        // loads that may still be in flight into this CTA's shared memory: wait for them, bounded
        for (int j = 0; j < stages; ++j) {
            const int jt = it + j;
            (void)mbar_wait_bounded(&full_bar[jt % stages], static_cast<unsigned>(jt / stages) & 1u, 100000000ull);
        }
    }
}

// Self-test of the bounded wait: a barrier that nobody ever arrives on.  Every thread's wait must
// give up after `limit_ns` and the kernel must record kStatusTimeout and return.  No memory is
// touched besides the status word.
__global__ void __launch_bounds__(kThreads)
bounded_wait_selftest_kernel(int* __restrict__ status, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool ok = mbar_wait_bounded(&bar, 0u, limit_ns);
    if (__syncthreads_or(ok ? 0 : 1) && threadIdx.x == 0) atomicOr(status, kStatusTimeout);
}

}  // namespace grawa
