// Host side of libgrawa: argument validation, the cached work-list plan, kernel launches and
// the C ABI declared in include/grawa.h.  There is no CPU implementation of the update here.
#include "../../include/grawa.h"

#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <memory>
#include <mutex>
#include <string>
#include <vector>

#include "kernels.cuh"
#include "center_pull_bulk.cuh"
#include "kernels_16bit.cuh"
#include "center_pull_staged_any.cuh"

namespace grawa {

static_assert(kMaxWorkers == GRAWA_MAX_WORKERS, "header and kernels disagree on the worker limit");

// ------------------------------------------------------------------ process-wide state
static std::mutex g_mutex;
static std::atomic<int64_t> g_launches{0};
static int64_t g_sumsq_tile = 8192;
static int64_t g_pull_tile = 0;           // 0 = one pass of the register kernel, pull_pass_elems(M)
static int64_t g_pull_variant = 0;
static int64_t g_bulk_tile = 0;           // 0 = chosen from M so that at least three stages fit
static int64_t g_kernel_timing = 0;
static int64_t g_pdl = 1;
static int64_t g_pull_preload = 1;
static int64_t g_pull_wide = 1;             // fp32 register kernel: 32-byte accesses when every base is 32-byte aligned
static int64_t g_pull16_staged = 1;         // 16-bit storage, 5..16 workers: shared-memory staged kernel (1) or register kernel (0)
static int64_t g_pull_prefetch_waves = 3;
static int64_t g_sumsq_prefetch_waves = 1;
static int64_t g_sumsq_ctas_per_sm = 0;   // 0 = one CTA per work item
static int64_t g_pull_ctas_per_sm = 0;    // 0 = one CTA per work item
static thread_local std::string t_cuda_error;

static grawa_status cuda_fail(cudaError_t err, const char* what)
{
    char buf[512];
    std::snprintf(buf, sizeof buf, "%s: %s (%s)", what, cudaGetErrorString(err), cudaGetErrorName(err));
    t_cuda_error = buf;
    return GRAWA_ERR_CUDA;
}

#define GRAWA_CUDA_TRY(expr)                                        \
    do {                                                            \
        cudaError_t err__ = (expr);                                 \
        if (err__ != cudaSuccess) return cuda_fail(err__, #expr);   \
    } while (0)

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Dynamic shared memory the bulk-copy centre+pull kernel may use (one CTA per SM).
constexpr size_t kBulkSmemBudget = 200 * 1024;

// Does the centre+pull of an M-worker problem take the bulk-copy kernel?  (Only when asked for: the staged
// kernels replaced it as the vector path for more than 16 workers.)
static bool wants_bulk(int) { return g_pull_variant == 2; }

// Elements per slice of a bulk-copy stage: the option, or the largest multiple of 256 up to 4096
// that leaves room for three stages of M+1 slices.
static int64_t bulk_tile_for(int M)
{
    if (g_bulk_tile > 0) return g_bulk_tile;
    const int64_t fit = static_cast<int64_t>(kBulkSmemBudget / (3 * sizeof(float) * (static_cast<size_t>(M) + 1)));
    return std::max<int64_t>(256, std::min<int64_t>(4096, fit / 256 * 256));
}

// ------------------------------------------------------------------ work list
// Tile used inside one layer: `tile`, doubled until the layer has at most `max_items` items (0 =
// no limit).  Bounds the number of atomic additions that meet on one row of exact sums for a huge
// layer, without giving up the fine grain that balances the many small layers.
static int64_t layer_tile(int64_t layer_elems, int64_t tile, int64_t max_items)
{
    int64_t t = tile;
    while (max_items > 0 && layer_elems / t > max_items && t < (int64_t{1} << 28)) t *= 2;
    return t;
}

constexpr int64_t kMaxSumsqItemsPerLayer = 1024;

// Cuts every non-empty layer at the absolute multiples of its tile that fall inside it.
static void build_segments(const std::vector<int64_t>& off, int64_t tile, int64_t max_items, std::vector<Segment>* segs)
{
    const int K = static_cast<int>(off.size()) - 1;
    for (int k = 0; k < K; ++k) {
        int64_t pos = off[k];
        const int64_t end = off[k + 1];
        const int64_t t = layer_tile(end - pos, tile, max_items);
        while (pos < end) {
            const int64_t next = std::min(end, (pos / t + 1) * t);
            segs->push_back(Segment{pos, static_cast<int>(next - pos), k});
            pos = next;
        }
    }
}

// Scratch layout (all offsets 256-byte aligned).
struct WorkspaceLayout {
    size_t words, bins, state_end, S, A, beta, total;
};

// The first `state_end` bytes carry state from one step to the next (which copy of the digit rows
// is clean) and must start out as zeros; the rest is overwritten before it is read.
static WorkspaceLayout workspace_layout(int K, int M)
{
    WorkspaceLayout w{};
    size_t p = 0;
    w.words = p;    p = align_up(p + 256, 256);   // ints: [0] next_buf, [1] status, [2] work counter (unsigned)
    w.bins = p;     p = align_up(p + sizeof(unsigned long long) * 2 * static_cast<size_t>(K) * M * kRowWords, 256);
    w.state_end = p;
    w.S = p;        p = align_up(p + sizeof(double) * static_cast<size_t>(K) * M, 256);
    w.A = p;        p = align_up(p + sizeof(double) * (static_cast<size_t>(K) + 1) * M, 256);   // K rows of terms + scores
    w.beta = p;     p = align_up(p + sizeof(float) * static_cast<size_t>(K) * M, 256);
    w.total = p;
    return w;
}

struct Plan {
    int device = 0;
    cudaStream_t stream = nullptr;
    int64_t n = 0;
    int M = 0, K = 0;
    std::vector<int64_t> off;
    int64_t tile1 = 0, tile2 = 0;
    int C1 = 0, C2 = 0;
    Segment* d_segs1 = nullptr;      // sum-of-squares items
    Segment* d_segs2 = nullptr;      // per-layer centre+pull items
    bool ws_dirty = false;           // a step failed half-way: the owned scratch is cleared before the next one
    int elem = 4;                    // bytes per stored element the work lists were cut for
    std::vector<const void*> seen_ptrs;   // the last pointer table that passed validation (params, grads, centre)
    void* d_ws = nullptr;            // owned scratch (used when the caller passes none)
    WorkspaceLayout ws{};
    void* d_stage = nullptr;         // owned staging for the host-buffer entry point
    int sm_count = 148;
    std::vector<Segment> h_segs2;    // host copy of the centre+pull items (chunking of the host-buffer path)
    cudaStream_t d2h_stream = nullptr;   // downloads of the host-buffer path
    std::vector<cudaEvent_t> events;     // chunk-done events of the host-buffer path
    bool bulk = false;               // centre+pull items are cut for the bulk-copy kernel
    ~Plan()
    {
        cudaFree(d_segs1); cudaFree(d_segs2); cudaFree(d_ws); cudaFree(d_stage);
        if (d2h_stream) cudaStreamDestroy(d2h_stream);
        for (cudaEvent_t ev : events) cudaEventDestroy(ev);
    }
};

struct PlanKey {
    int device; cudaStream_t stream; int64_t n; int M; int elem; std::vector<int64_t> off;
    bool operator<(const PlanKey& o) const
    {
        if (device != o.device) return device < o.device;
        if (elem != o.elem) return elem < o.elem;
        if (stream != o.stream) return stream < o.stream;
        if (n != o.n) return n < o.n;
        if (M != o.M) return M < o.M;
        return off < o.off;
    }
};

// Event quads recorded around the three phases of a step while "kernel_timing" is on.
struct TimedStep { cudaEvent_t e[4]; };
static auto& g_timed_pool = *new std::vector<TimedStep>;   // created once, reused
static size_t g_timed_used = 0;

// Heap-allocated and never destroyed: at process exit the CUDA runtime may already be gone.
static auto& g_plans = *new std::map<PlanKey, std::unique_ptr<Plan>>;
static Plan* g_recent_plan = nullptr;      // plan of the most recent step (fast path of step_entry)
static auto& g_last_status = *new std::map<std::pair<int, cudaStream_t>, int*>;   // (device, stream) -> status word

// `elem`: bytes per stored element (4, or 2 for 16-bit storage, whose kernels cover twice the
// elements per pass and therefore cut the work lists with twice the tile).
static grawa_status get_plan(int64_t n, int M, const std::vector<int64_t>& off, cudaStream_t stream, Plan** out, int elem = 4)
{
    int device = 0;
    GRAWA_CUDA_TRY(cudaGetDevice(&device));
    PlanKey key{device, stream, n, M, elem, off};
    auto it = g_plans.find(key);
    if (it != g_plans.end()) { *out = it->second.get(); return GRAWA_OK; }

    std::unique_ptr<Plan> p(new Plan);
    p->device = device; p->stream = stream; p->n = n; p->M = M; p->off = off; p->elem = elem;
    p->K = static_cast<int>(off.size()) - 1;
    p->bulk = elem == 4 && wants_bulk(M);
    p->tile1 = g_sumsq_tile * (4 / elem);
    p->tile2 = p->bulk ? bulk_tile_for(M)
               : (g_pull_tile > 0 ? g_pull_tile
                  : M > kMaxRegWorkers ? staged_any_threads(M) * (16 / elem)
                  : (elem == 2 ? ((M > 4 && g_pull16_staged) ? pull16s_pass_elems(std::min(M, kMaxRegWorkers)) : pull16_pass_elems(std::min(M, kMaxRegWorkers)))
                               : pull_pass_elems(std::min(M, kMaxRegWorkers))));
    GRAWA_CUDA_TRY(cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, device));
    std::vector<Segment> s1, s2;
    build_segments(off, p->tile1, kMaxSumsqItemsPerLayer, &s1);
    build_segments(off, p->tile2, 0, &s2);
    if (s1.size() * static_cast<size_t>(M) > 0x7fffffffull || s2.size() > 0x7fffffffull) return GRAWA_ERR_INVALID_ARG;
    p->C1 = static_cast<int>(s1.size()); p->C2 = static_cast<int>(s2.size());
    p->h_segs2 = s2;
    p->ws = workspace_layout(p->K, M);
    GRAWA_CUDA_TRY(cudaMalloc(&p->d_segs1, sizeof(Segment) * std::max<size_t>(1, s1.size())));
    GRAWA_CUDA_TRY(cudaMalloc(&p->d_segs2, sizeof(Segment) * std::max<size_t>(1, s2.size())));
    GRAWA_CUDA_TRY(cudaMemcpy(p->d_segs1, s1.data(), sizeof(Segment) * s1.size(), cudaMemcpyHostToDevice));
    GRAWA_CUDA_TRY(cudaMemcpy(p->d_segs2, s2.data(), sizeof(Segment) * s2.size(), cudaMemcpyHostToDevice));
    *out = p.get();
    g_plans[key] = std::move(p);
    return GRAWA_OK;
}

// ------------------------------------------------------------------ validation
static bool ranges_overlap(const void* a, const void* b, size_t bytes)
{
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + bytes && y < x + bytes;
}

// Buffers: non-NULL, aligned to their element size, and no overlap visible from the pointer ranges.
static grawa_status validate_pointers(float* const* params, const float* const* grads, int64_t n, int M,
                                      const float* center_out, size_t elem_size)
{
    const size_t bytes = static_cast<size_t>(n) * elem_size;
    const uintptr_t amask = elem_size - 1;          // buffers must be aligned to their element size
    for (int m = 0; m < M; ++m) {
        if (params[m] == nullptr || (grads && grads[m] == nullptr)) return GRAWA_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(params[m]) & amask) || (grads && (reinterpret_cast<uintptr_t>(grads[m]) & amask)))
            return GRAWA_ERR_INVALID_ARG;
    }
    if (reinterpret_cast<uintptr_t>(center_out) & amask) return GRAWA_ERR_INVALID_ARG;
    for (int a = 0; a < M; ++a) {
        for (int b = a + 1; b < M; ++b)
            if (ranges_overlap(params[a], params[b], bytes)) return GRAWA_ERR_INVALID_ARG;
        if (center_out && ranges_overlap(params[a], center_out, bytes)) return GRAWA_ERR_INVALID_ARG;
        if (grads) {
            for (int b = 0; b < M; ++b)
                if (ranges_overlap(params[a], grads[b], bytes)) return GRAWA_ERR_INVALID_ARG;
            if (center_out && ranges_overlap(grads[a], center_out, bytes)) return GRAWA_ERR_INVALID_ARG;
        }
    }
    return GRAWA_OK;
}

// Sizes, pull strength and the shape of the layer table (not its contents).
static grawa_status validate_scalars(const void* params, int64_t n, int M, float pull, const int64_t* layer_offsets, int n_layers)
{
    if (M < 1 || M > GRAWA_MAX_WORKERS || n < 0 || n_layers < 0) return GRAWA_ERR_INVALID_ARG;
    if (!(pull >= 0.0f && pull <= 1.0f)) return GRAWA_ERR_INVALID_ARG;   // also rejects NaN
    if (params == nullptr) return GRAWA_ERR_INVALID_ARG;
    if ((layer_offsets == nullptr) != (n_layers == 0)) return GRAWA_ERR_INVALID_ARG;
    return GRAWA_OK;
}

static grawa_status validate(float* const* params, const float* const* grads, int64_t n, int M, float pull,
                             const int64_t* layer_offsets, int n_layers, const float* center_out,
                             std::vector<int64_t>* off, size_t elem_size = sizeof(float))
{
    const grawa_status st = validate_scalars(params, n, M, pull, layer_offsets, n_layers);
    if (st != GRAWA_OK) return st;
    if (layer_offsets) {
        if (layer_offsets[0] != 0 || layer_offsets[n_layers] != n) return GRAWA_ERR_INVALID_ARG;
        for (int k = 0; k < n_layers; ++k)
            if (layer_offsets[k + 1] < layer_offsets[k]) return GRAWA_ERR_INVALID_ARG;
        off->assign(layer_offsets, layer_offsets + n_layers + 1);
    } else {
        off->assign({0, n});
    }
    if (n == 0) return GRAWA_OK;
    return validate_pointers(params, grads, n, M, center_out, elem_size);
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline bool dtype_ok(grawa_dtype d) { return d == GRAWA_F32 || d == GRAWA_BF16 || d == GRAWA_F16; }
static inline bool variant_ok(grawa_variant v)
{
    return v == GRAWA_VARIANT_GRAWA || v == GRAWA_VARIANT_MGRAWA || v == GRAWA_VARIANT_LGRAWA;
}
static inline size_t elem_size(int dtype) { return dtype == 0 ? sizeof(float) : size_t{2}; }

// ------------------------------------------------------------------ launches
// One launch, optionally with programmatic stream serialisation (the kernel may start launching
// while its predecessor on the stream drains; it waits for it in grid_dependency_sync()).
template <typename... KArgs, typename... Args>
static cudaError_t launch_kernel_smem(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t stream, bool pdl,
                                      Args&&... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(static_cast<unsigned>(block));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    ++g_launches;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename... KArgs, typename... Args>
static cudaError_t launch_kernel(void (*kernel)(KArgs...), int grid, int block, cudaStream_t stream, bool pdl, Args&&... args)
{
    return launch_kernel_smem(kernel, grid, block, 0, stream, pdl, static_cast<Args&&>(args)...);
}

// Bulk-copy centre+pull: MT = M for 2..16 (register column), MT = 0 for larger M.

template <int MT>
static cudaError_t launch_center_pull_bulk(bool per_layer, int grid, int item_begin, int item_end, size_t smem, cudaStream_t stream,
                                           bool pdl, const MutPtrs& x, float* center, const float* beta, const Segment* segs,
                                           long long n, int tile, int stages, int M, float pull, unsigned* counter, int* status)
{
    auto kernel = per_layer ? center_pull_bulk_kernel<MT, true> : center_pull_bulk_kernel<MT, false>;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kBulkSmemBudget));
    if (err != cudaSuccess) return err;
    return launch_kernel_smem(kernel, grid, kThreads, smem, stream, pdl, x, center, beta, segs, item_begin, item_end, n, tile, stages,
                              M, pull, counter, status);
}

template <int MT>
struct CenterPullBulkDispatch {
    template <typename... A>
    static cudaError_t run(int m, A&&... a)
    {
        if (m == MT) return launch_center_pull_bulk<MT>(static_cast<A&&>(a)...);
        return CenterPullBulkDispatch<MT - 1>::run(m, static_cast<A&&>(a)...);
    }
};
template <>
struct CenterPullBulkDispatch<1> {
    template <typename... A>
    static cudaError_t run(int, A&&... a)
    {
        return launch_center_pull_bulk<0>(static_cast<A&&>(a)...);
    }
};

template <int M>
static cudaError_t launch_center_pull(bool per_layer, bool wide, int grid, int item_begin, int item_end, cudaStream_t stream, bool pdl,
                                      const MutPtrs& x, float* center, const float* beta, const Segment* segs, long long n, int tile,
                                      float pull, int preload, int prefetch_stride, int prefetch_waves)
{
    // `wide`: every base is 32-byte aligned, so the columns are moved by 32-byte loads and stores
    auto kernel = wide ? (per_layer ? center_pull_kernel<M, true, 8> : center_pull_kernel<M, false, 8>)
                       : (per_layer ? center_pull_kernel<M, true, 4> : center_pull_kernel<M, false, 4>);
    return launch_kernel(kernel, grid, wide ? pull_threads(M, 8) : pull_threads(M, 4), stream, pdl, x, center, beta, segs, item_begin,
                         item_end, n, tile, pull, 1, preload, prefetch_stride, prefetch_waves);
}

template <int M>
struct CenterPullDispatch {
    template <typename... A>
    static cudaError_t run(int m, A&&... a)
    {
        if (m == M) return launch_center_pull<M>(static_cast<A&&>(a)...);
        return CenterPullDispatch<M - 1>::run(m, static_cast<A&&>(a)...);
    }
};
template <>
struct CenterPullDispatch<1> {
    template <typename... A>
    static cudaError_t run(int, A&&...)
    {
        return cudaErrorInvalidValue;
    }
};

// 16-bit storage: register kernel for 2..16 aligned workers.
template <typename T, int M>
static cudaError_t launch_center_pull16(bool per_layer, bool wide, int grid, int item_begin, int item_end, cudaStream_t stream, bool pdl,
                                        const MutPtrs& x, T* center, const float* beta, const Segment* segs, long long n,
                                        int tile, float pull)
{
    constexpr bool kCanWide = M <= 4;               // 32-byte columns: up to 4 workers
    auto kernel = (wide && kCanWide) ? (per_layer ? center_pull16_kernel<T, M, true, kCanWide> : center_pull16_kernel<T, M, false, kCanWide>)
                                     : (per_layer ? center_pull16_kernel<T, M, true, false> : center_pull16_kernel<T, M, false, false>);
    return launch_kernel(kernel, grid, kThreads, stream, pdl, x, center, beta, segs, item_begin, item_end, n, tile, pull, 1);
}

template <typename T, int M>
struct CenterPull16Dispatch {
    template <typename... A>
    static cudaError_t run(int m, A&&... a)
    {
        if (m == M) return launch_center_pull16<T, M>(static_cast<A&&>(a)...);
        return CenterPull16Dispatch<T, M - 1>::run(m, static_cast<A&&>(a)...);
    }
};
template <typename T>
struct CenterPull16Dispatch<T, 1> {
    template <typename... A>
    static cudaError_t run(int, A&&...)
    {
        return cudaErrorInvalidValue;
    }
};

// 16-bit storage, 5..16 aligned workers: columns staged through shared memory by per-thread asynchronous copies.
template <typename T, int M>
static cudaError_t launch_center_pull16_staged(bool per_layer, int grid, int item_begin, int item_end, cudaStream_t stream, bool pdl,
                                               const MutPtrs& x, T* center, const float* beta, const Segment* segs, long long n,
                                               int tile, float pull, int preload)
{
    const size_t smem = sizeof(uint4) * static_cast<size_t>(M) * kThreads * pull16s_cols(M);
    auto kernel = per_layer ? center_pull16_staged_kernel<T, M, true> : center_pull16_staged_kernel<T, M, false>;
    const cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (err != cudaSuccess) return err;
    return launch_kernel_smem(kernel, grid, kThreads, smem, stream, pdl, x, center, beta, segs, item_begin, item_end, n, tile, pull,
                              preload);
}

template <typename T, int M>
struct CenterPull16StagedDispatch {
    template <typename... A>
    static cudaError_t run(int m, A&&... a)
    {
        if (m == M) return launch_center_pull16_staged<T, M>(static_cast<A&&>(a)...);
        return CenterPull16StagedDispatch<T, M - 1>::run(m, static_cast<A&&>(a)...);
    }
};
template <typename T>
struct CenterPull16StagedDispatch<T, 4> {
    template <typename... A>
    static cudaError_t run(int, A&&...)
    {
        return cudaErrorInvalidValue;
    }
};

// More than 16 aligned workers, any storage type: the staged kernel with a run-time worker count.
template <typename T>
static cudaError_t launch_center_pull_staged_any(bool per_layer, int grid, int item_begin, int item_end, cudaStream_t stream, bool pdl,
                                                 const MutPtrs& x, T* center, const float* beta, const Segment* segs, long long n,
                                                 int tile, float pull, int M, int preload)
{
    const int threads = staged_any_threads(M);
    const size_t smem = align_up(sizeof(uint4) * static_cast<size_t>(M) * threads + sizeof(float) * M, 16);
    auto kernel = per_layer ? center_pull_staged_any_kernel<T, true> : center_pull_staged_any_kernel<T, false>;
    const cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024);
    if (err != cudaSuccess) return err;
    return launch_kernel_smem(kernel, grid, threads, smem, stream, pdl, x, center, beta, segs, item_begin, item_end, n, tile, pull, M,
                              preload);
}

// Device pointers and launch facts of one step, resolved once from the plan and the options.
struct StepContext {
    Plan* plan = nullptr;
    int variant = 0, M = 0;
    int64_t n = 0;
    float pull = 0.f;
    cudaStream_t stream = nullptr;
    ConstPtrs gp{};
    MutPtrs xp{};
    float* center = nullptr;
    bool vec_g = true, vec_x = true, pdl = false;
    bool wide_x = true;            // parameters and centre are 32-byte aligned as well
    StepScratch sc{};
    int* status = nullptr;
    unsigned* counter = nullptr;
    TimedStep* ts = nullptr;
    int pull_items = 0;            // centre+pull work items of the whole vector
    int dtype = 0;                 // storage of params / grads / centre: 0 fp32, 1 bfloat16, 2 half
    bool preload = false;          // centre+pull may load parameters before its dependency wait (see the kernel)
};

static grawa_status make_context(int variant, float* const* params, const float* const* grads, int64_t n, int M, float pull,
                                 float* center_out, const grawa_options* opt, cudaStream_t stream, Plan* plan, StepContext* ctx)
{
    const int K = plan->K;
    char* ws = static_cast<char*>(opt ? opt->workspace : nullptr);
    if (ws) {
        if ((reinterpret_cast<uintptr_t>(ws) & 255u) || opt->workspace_bytes < plan->ws.total) return GRAWA_ERR_WORKSPACE;
    } else {
        if (opt && opt->workspace_bytes != 0) return GRAWA_ERR_WORKSPACE;
        if (!plan->d_ws) {
            GRAWA_CUDA_TRY(cudaMalloc(&plan->d_ws, plan->ws.total));
            plan->ws_dirty = true;
        }
        ws = static_cast<char*>(plan->d_ws);
    }
    // The state part of the scratch must be zero when a step starts from scratch: always for a
    // caller's buffer (its contents are the caller's business between calls), and for the plan's own
    // buffer when it is new or a step was abandoned half-way.
    if (ws != plan->d_ws || plan->ws_dirty) {
        GRAWA_CUDA_TRY(cudaMemsetAsync(ws, 0, plan->ws.state_end, stream));
        if (ws == plan->d_ws) plan->ws_dirty = false;
    }
    ctx->plan = plan; ctx->variant = variant; ctx->M = M; ctx->n = n; ctx->pull = pull; ctx->stream = stream;
    ctx->center = center_out;
    ctx->status = reinterpret_cast<int*>(ws + plan->ws.words) + 1;
    ctx->counter = reinterpret_cast<unsigned*>(ws + plan->ws.words) + 2;
    g_last_status[{plan->device, stream}] = ctx->status;
    ctx->vec_g = true;
    ctx->vec_x = center_out == nullptr || aligned16(center_out);
    ctx->wide_x = (reinterpret_cast<uintptr_t>(center_out) & 31u) == 0;
    for (int m = 0; m < M; ++m) {
        ctx->gp.p[m] = grads ? grads[m] : nullptr; ctx->xp.p[m] = params[m];
        ctx->vec_g = ctx->vec_g && grads && aligned16(grads[m]);
        ctx->vec_x = ctx->vec_x && aligned16(params[m]);
        ctx->wide_x = ctx->wide_x && (reinterpret_cast<uintptr_t>(params[m]) & 31u) == 0;
    }
    StepScratch& sc = ctx->sc;
    sc.segs = plan->d_segs1;
    sc.C = plan->C1; sc.K = K; sc.M = M; sc.variant = variant; sc.n = n;
    sc.prefetch_stride = 0; sc.prefetch_waves = 0;
    sc.bins = reinterpret_cast<unsigned long long*>(ws + plan->ws.bins);
    sc.next_buf = reinterpret_cast<int*>(ws + plan->ws.words);
    sc.S = reinterpret_cast<double*>(ws + plan->ws.S);
    sc.A = reinterpret_cast<double*>(ws + plan->ws.A);
    sc.beta = reinterpret_cast<float*>(ws + plan->ws.beta);
    sc.status_copy = opt ? opt->status_word : nullptr;
    sc.status = ctx->status; sc.work_counter = ctx->counter;
    sc.weights_out = opt ? opt->weights_out : nullptr;
    sc.scores_out = opt ? opt->scores_out : nullptr;
    sc.sumsq_out = opt ? opt->sumsq_out : nullptr;
    sc.given = nullptr; sc.given_parts = 1; sc.given_sums = 0;
    const int64_t tiles = variant == kLgrawa ? plan->C2 : (n + plan->tile2 - 1) / plan->tile2;
    if (tiles > 0x7fffffffll) return GRAWA_ERR_INVALID_ARG;
    ctx->pull_items = static_cast<int>(tiles);
    ctx->ts = nullptr;
    ctx->pdl = g_pdl != 0;
    return GRAWA_OK;
}

// Steps 2-3.  LGRAWA: one warp per layer in as many CTAs as that takes.  One weight per worker: one
// CTA with a thread per (layer, worker) row when that fits, runs of rows per thread up to
// kFinSharedOutRows rows, beyond that the rows shared out over several full CTAs.
static cudaError_t launch_finalize(const StepContext& c)
{
    const Plan* plan = c.plan;
    const int64_t rows = static_cast<int64_t>(plan->K) * c.M;
    int grid = 1, block = static_cast<int>(std::max<int64_t>(128, std::min<int64_t>(kFinThreadsFlat, (rows + 31) / 32 * 32)));
    if (c.variant == kLgrawa && c.sc.given == nullptr) {
        block = kFinThreadsLayered;
        grid = std::max(1, std::min((plan->K + block / 32 - 1) / (block / 32), 4 * plan->sm_count));
    } else if (c.variant == kLgrawa) {
        // given scores: no sum-of-squares kernel has cleared the status words, and several CTAs only
        // add their flags to them, so they are cleared here when the layers take more than one CTA
        if (plan->K > kFinGivenLayersOneCta) {
            block = kFinThreadsFlat;
            grid = std::min((plan->K + block / 32 - 1) / (block / 32), 4 * plan->sm_count);
            cudaError_t err = cudaMemsetAsync(c.sc.status, 0, sizeof(int), c.stream);
            if (err == cudaSuccess && c.sc.status_copy) err = cudaMemsetAsync(c.sc.status_copy, 0, sizeof(int), c.stream);
            if (err != cudaSuccess) return err;
        }
    } else if (rows > kFinSharedOutRows) {
        grid = static_cast<int>(std::min<int64_t>((rows + kFinThreadsFlat - 1) / kFinThreadsFlat, plan->sm_count));
    }
    return launch_kernel(finalize_kernel, grid, block, c.stream, c.pdl, c.sc);
}

// Steps 1-3: sums of squares, scores, weights (two launches).
static grawa_status enqueue_weights_launches(StepContext& c);
static grawa_status enqueue_weights(StepContext& c)
{
    const grawa_status st = enqueue_weights_launches(c);
    if (st != GRAWA_OK) c.plan->ws_dirty = true;       // the two copies of the digit rows may be out of step
    return st;
}

static grawa_status enqueue_weights_launches(StepContext& c)
{
    Plan* plan = c.plan;
    if (c.sc.given != nullptr) {                     // scores are given: no pass over gradients
        if (c.ts) GRAWA_CUDA_TRY(cudaEventRecord(c.ts->e[1], c.stream));
        GRAWA_CUDA_TRY(launch_finalize(c));
        if (c.ts) GRAWA_CUDA_TRY(cudaEventRecord(c.ts->e[2], c.stream));
        return GRAWA_OK;
    }
    const int items1 = plan->C1 * c.M;
    const int grid1 = g_sumsq_ctas_per_sm > 0
                          ? static_cast<int>(std::min<int64_t>(items1, g_sumsq_ctas_per_sm * plan->sm_count)) : items1;
    const int vg = c.vec_g ? 1 : 0;
    c.sc.prefetch_stride = 6 * plan->sm_count;           // CTAs resident at the start of the kernel
    c.sc.prefetch_waves = (grid1 <= 64 * c.sc.prefetch_stride) ? static_cast<int>(g_sumsq_prefetch_waves) : 0;
    if (c.dtype == 1)
        GRAWA_CUDA_TRY(launch_kernel(sumsq16_kernel<__nv_bfloat16, 8>, grid1, kThreads, c.stream, c.pdl, c.gp, c.sc, items1, vg));
    else if (c.dtype == 2)
        GRAWA_CUDA_TRY(launch_kernel(sumsq16_kernel<__half, 8>, grid1, kThreads, c.stream, c.pdl, c.gp, c.sc, items1, vg));
    else
        GRAWA_CUDA_TRY(launch_kernel(sumsq_kernel<8>, grid1, kThreads, c.stream, c.pdl, c.gp, c.sc, items1, vg));
    if (c.ts) GRAWA_CUDA_TRY(cudaEventRecord(c.ts->e[1], c.stream));
    GRAWA_CUDA_TRY(launch_finalize(c));
    if (c.ts) GRAWA_CUDA_TRY(cudaEventRecord(c.ts->e[2], c.stream));
    return GRAWA_OK;
}

// Steps 4-5 on 16-bit storage: register kernel for 2..16 aligned workers, scalar kernel otherwise.
template <typename T>
static grawa_status enqueue_center_pull16_t(StepContext& c, int item_begin, int item_end)
{
    Plan* plan = c.plan;
    const int M = c.M;
    const bool per_layer = c.variant == kLgrawa;
    const int grid = item_end - item_begin;
    const int tile = static_cast<int>(plan->tile2);
    T* center = reinterpret_cast<T*>(c.center);
    if (c.vec_x && M > 4 && M <= kMaxRegWorkers && g_pull16_staged) {
        GRAWA_CUDA_TRY((CenterPull16StagedDispatch<T, kMaxRegWorkers>::run(M, per_layer, grid, item_begin, item_end, c.stream, c.pdl,
                                                                           c.xp, center, c.sc.beta, plan->d_segs2, c.n, tile, c.pull,
                                                                           (c.preload && g_pull_preload) ? 1 : 0)));
    } else if (c.vec_x && M > kMaxRegWorkers) {
        GRAWA_CUDA_TRY(launch_center_pull_staged_any<T>(per_layer, grid, item_begin, item_end, c.stream, c.pdl, c.xp, center, c.sc.beta,
                                                        plan->d_segs2, c.n, tile, c.pull, M, (c.preload && g_pull_preload) ? 1 : 0));
    } else if (c.vec_x && M <= kMaxRegWorkers) {
        GRAWA_CUDA_TRY((CenterPull16Dispatch<T, kMaxRegWorkers>::run(M, per_layer, c.wide_x && g_pull_wide, grid, item_begin, item_end, c.stream, c.pdl, c.xp,
                                                                     center, c.sc.beta, plan->d_segs2, c.n, tile, c.pull)));
    } else {
        GRAWA_CUDA_TRY(launch_kernel(center_pull16_generic_kernel<T>, grid, kThreads, c.stream, c.pdl, c.xp, center, c.sc.beta,
                                     plan->d_segs2, per_layer ? 1 : 0, item_begin, c.n, tile, c.pull, M));
    }
    return GRAWA_OK;
}

static grawa_status enqueue_center_pull16(StepContext& c, int item_begin, int item_end)
{
    if (c.dtype == 1) return enqueue_center_pull16_t<__nv_bfloat16>(c, item_begin, item_end);
    return enqueue_center_pull16_t<__half>(c, item_begin, item_end);
}

// Steps 4-5 on the work items [item_begin, item_end) (one launch).  M >= 2.
static grawa_status enqueue_center_pull(StepContext& c, int item_begin, int item_end)
{
    Plan* plan = c.plan;
    const int M = c.M;
    const bool per_layer = c.variant == kLgrawa;
    const int grid = item_end - item_begin;
    if (grid <= 0) return GRAWA_OK;
    const int tile = static_cast<int>(plan->tile2);
    const float* beta = c.sc.beta;
    if (c.dtype != 0) return enqueue_center_pull16(c, item_begin, item_end);
    // bulk-copy variant: only when asked for
    const size_t stage_bytes = sizeof(float) * static_cast<size_t>(plan->tile2) * (M + 1);
    const int stages = static_cast<int>(std::min<size_t>(kBulkMaxStages, kBulkSmemBudget / stage_bytes));
    if (c.vec_x && plan->bulk && stages >= 2) {
        const int gridb = std::min(grid, plan->sm_count);
        GRAWA_CUDA_TRY(CenterPullBulkDispatch<kMaxRegWorkers>::run(M <= kMaxRegWorkers ? M : 1, per_layer, gridb, item_begin, item_end,
                                                                   stage_bytes * stages, c.stream, c.pdl, c.xp, c.center, beta,
                                                                   plan->d_segs2, c.n, tile, stages, M, c.pull, c.counter, c.status));
    } else if (c.vec_x && M > kMaxRegWorkers) {
        GRAWA_CUDA_TRY(launch_center_pull_staged_any<float>(per_layer, grid, item_begin, item_end, c.stream, c.pdl, c.xp, c.center, beta,
                                                            plan->d_segs2, c.n, tile, c.pull, M, (c.preload && g_pull_preload) ? 1 : 0));
    } else if (c.vec_x && M <= kMaxRegWorkers) {
        // L2 prefetch of later items during the weights' finalisation: pays on short steps only (a few
        // dozen waves of CTAs); on long ones the window it fills is negligible and the hint costs a little
        const int stride = 2 * plan->sm_count;
        const int waves = (grid <= 64 * stride) ? static_cast<int>(g_pull_prefetch_waves) : 0;
        const int grid2 = g_pull_ctas_per_sm > 0
                              ? static_cast<int>(std::min<int64_t>(grid, g_pull_ctas_per_sm * plan->sm_count)) : grid;
        GRAWA_CUDA_TRY(CenterPullDispatch<kMaxRegWorkers>::run(M, per_layer, c.wide_x && g_pull_wide, grid2, item_begin, item_end, c.stream, c.pdl, c.xp,
                                                               c.center, beta, plan->d_segs2, c.n, tile, c.pull,
                                                               (c.preload && g_pull_preload) ? 1 : 0, stride, waves));
    } else {
        GRAWA_CUDA_TRY(launch_kernel(center_pull_generic_kernel, grid, kThreads, c.stream, c.pdl, c.xp, c.center, beta, plan->d_segs2,
                                     per_layer ? 1 : 0, item_begin, c.n, tile, c.pull, M));
    }
    return GRAWA_OK;
}

// Given scores of a step that reads no gradients: per-layer norms, or `parts` sets of per-layer sums.
struct GivenScores {
    const double* data = nullptr;
    int parts = 1;
    int sums = 0;
};

static grawa_status enqueue_step(int variant, float* const* params, const float* const* grads, const GivenScores& given,
                                 int64_t n, int M, float pull, float* center_out, const grawa_options* opt,
                                 cudaStream_t stream, Plan* plan, int dtype = 0)
{
    StepContext c;
    grawa_status st = make_context(variant, params, grads, n, M, pull, center_out, opt, stream, plan, &c);
    if (st != GRAWA_OK) return st;
    c.dtype = dtype;
    c.sc.given = given.data; c.sc.given_parts = given.parts; c.sc.given_sums = given.sums;
    if (g_kernel_timing) {
        if (g_timed_used == g_timed_pool.size()) {
            TimedStep fresh{};
            for (auto& ev : fresh.e) GRAWA_CUDA_TRY(cudaEventCreate(&ev));
            g_timed_pool.push_back(fresh);
        }
        c.ts = &g_timed_pool[g_timed_used++];
        c.pdl = false;                               // event records between the kernels need plain ordering
        GRAWA_CUDA_TRY(cudaEventRecord(c.ts->e[0], stream));
    }
    st = enqueue_weights(c);
    if (st != GRAWA_OK) return st;
    if (M == 1) {
        if (center_out) {
            const bool v = aligned16(center_out) && aligned16(params[0]);
            const int grid = static_cast<int>(std::min<int64_t>((n + kThreads * 4 - 1) / (kThreads * 4), 148 * 16));
            if (dtype == 1)
                GRAWA_CUDA_TRY(launch_kernel(copy16_kernel<__nv_bfloat16>, grid, kThreads, stream, c.pdl,
                                             reinterpret_cast<const __nv_bfloat16*>(params[0]),
                                             reinterpret_cast<__nv_bfloat16*>(center_out), n));
            else if (dtype == 2)
                GRAWA_CUDA_TRY(launch_kernel(copy16_kernel<__half>, grid, kThreads, stream, c.pdl,
                                             reinterpret_cast<const __half*>(params[0]), reinterpret_cast<__half*>(center_out), n));
            else
                GRAWA_CUDA_TRY(launch_kernel(copy_kernel, grid, kThreads, stream, c.pdl, params[0], center_out, n, v ? 1 : 0));
        }
    } else {
        c.preload = true;          // the kernels in front of it on the stream are this step's own
        st = enqueue_center_pull(c, 0, c.pull_items);
        if (st != GRAWA_OK) return st;
    }
    if (c.ts) GRAWA_CUDA_TRY(cudaEventRecord(c.ts->e[3], stream));
    return GRAWA_OK;
}

static grawa_status step_entry(int variant, float* const* params, const float* const* grads, const GivenScores& given,
                               int64_t n, int M, float pull, const int64_t* layer_offsets, int n_layers, float* center_out,
                               const grawa_options* opt, cudaStream_t stream, int dtype = 0)
{
    if ((grads == nullptr) == (given.data == nullptr)) return GRAWA_ERR_INVALID_ARG;   // exactly one source of scores
    if (given.parts < 1) return GRAWA_ERR_INVALID_ARG;
    const int elem = dtype == 0 ? 4 : 2;
    grawa_status st = validate_scalars(params, n, M, pull, layer_offsets, n_layers);
    if (st != GRAWA_OK) return st;
    std::lock_guard<std::mutex> lock(g_mutex);
    // Fast path of a training loop: the same problem as the call before (device, stream, sizes and a
    // byte-identical layer table), usually with the same buffers.  The table was validated when the
    // plan was built and the buffers when they were first seen, so neither is walked again.
    Plan* plan = g_recent_plan;
    bool same_problem =
        n > 0 && plan != nullptr && plan->stream == stream && plan->n == n && plan->M == M && plan->elem == elem &&
        (layer_offsets ? (plan->K == n_layers && std::memcmp(plan->off.data(), layer_offsets, sizeof(int64_t) * (static_cast<size_t>(n_layers) + 1)) == 0)
                       : plan->K == 1);
    if (same_problem) {
        int device = 0;
        GRAWA_CUDA_TRY(cudaGetDevice(&device));
        same_problem = plan->device == device;
    }
    if (!same_problem) {
        std::vector<int64_t> off;
        st = validate(params, grads, n, M, pull, layer_offsets, n_layers, center_out, &off, static_cast<size_t>(elem));
        if (st != GRAWA_OK || n == 0) return st;
        st = get_plan(n, M, off, stream, &plan, elem);
        if (st != GRAWA_OK) return st;
        plan->seen_ptrs.clear();
        g_recent_plan = plan;
    }
    // the pointer table: 2M + 1 addresses; byte-identical to the last validated one = nothing to check
    const void* ptrs[2 * GRAWA_MAX_WORKERS + 1];
    for (int m = 0; m < M; ++m) { ptrs[m] = params[m]; ptrs[M + m] = grads ? grads[m] : nullptr; }
    ptrs[2 * M] = center_out;
    const size_t np = 2 * static_cast<size_t>(M) + 1;
    if (plan->seen_ptrs.size() != np || std::memcmp(plan->seen_ptrs.data(), ptrs, sizeof(void*) * np) != 0) {
        st = validate_pointers(params, grads, n, M, center_out, static_cast<size_t>(elem));
        if (st != GRAWA_OK) return st;
        plan->seen_ptrs.assign(ptrs, ptrs + np);
    }
    return enqueue_step(variant, params, grads, given, n, M, pull, center_out, opt, stream, plan, dtype);
}

// ------------------------------------------------------------------ allocation-free sum of squares
// Scratch that lives in the library image instead of in an allocation: one array per GPU that
// loads the library, held until the process exits.  In host code `g_static_partials` is only a
// handle for cudaGetSymbolAddress; kernels are given the address that call returns.
constexpr int kStaticTile = 16384;
static_assert(kStaticTile % 4 == 0, "tiles must keep 16-byte alignment");
static __device__ __align__(256) double g_static_partials[GRAWA_STATIC_MAX_PARTIALS];

constexpr int kMaxDevices = 64;
static double* g_static_partials_addr[kMaxDevices] = {};   // per device, filled on first use

// Variant of sumsq_kernel for one flat layer: items are (worker, tile of `tile` elements) found
// by arithmetic, so no work list has to exist in device memory.
template <int UNROLL>
__global__ void __launch_bounds__(kThreads)
sumsq_flat_kernel(ConstPtrs grads, long long n, int tiles, int tile, double* __restrict__ partials, int vec_ok)
{
    const int item = blockIdx.x;
    const int m = item / tiles;
    const int t = item - m * tiles;
    const float* __restrict__ g = grads.p[m];
    const long long b = static_cast<long long>(t) * tile, e = min(n, b + tile);
    const int tid = threadIdx.x;
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
            v[u] = (c < ncol && in_bounds(hb + 4LL * c, 4, b, e, n)) ? ld_stream4(g4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
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
        const double v = in_bounds(i, 1, b, e, n) ? static_cast<double>(ld_stream1(g + i)) : 0.0;
        dacc += v * v;
    }
    for (long long i = te + tid; i < e; i += kThreads) {
        const double v = in_bounds(i, 1, b, e, n) ? static_cast<double>(ld_stream1(g + i)) : 0.0;
        dacc += v * v;
    }
    const double total = block_sum_fixed_order<kThreads>(dacc);
    if (tid == 0 && scratch_ok(static_cast<long long>(m) * tiles + t, GRAWA_STATIC_MAX_PARTIALS))
        partials[static_cast<size_t>(m) * tiles + t] = total;
}

// One CTA per worker adds that worker's `tiles` partial sums in a fixed order.
__global__ void __launch_bounds__(kFinalizeThreads)
sum_partials_kernel(const double* __restrict__ partials, int tiles, double* __restrict__ out)
{
    const double* __restrict__ row = partials + static_cast<size_t>(blockIdx.x) * tiles;
    double acc = 0.0;
    for (int s = threadIdx.x; s < tiles; s += kFinalizeThreads)
        if (scratch_ok(static_cast<long long>(blockIdx.x) * tiles + s, GRAWA_STATIC_MAX_PARTIALS)) acc += row[s];
    const double total = block_sum_fixed_order<kFinalizeThreads>(acc);
    if (threadIdx.x == 0) out[blockIdx.x] = total;
}

}  // namespace grawa

using namespace grawa;

extern "C" {

int grawa_version(void) { return 100; }

const char* grawa_status_string(grawa_status status)
{
    switch (status) {
        case GRAWA_OK: return "ok";
        case GRAWA_ERR_INVALID_ARG: return "invalid argument";
        case GRAWA_ERR_CUDA: return "CUDA runtime error";
        case GRAWA_ERR_NONFINITE: return "non-finite gradient score";
        case GRAWA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case GRAWA_ERR_TIMEOUT: return "bounded device wait ran out";
        case GRAWA_ERR_TOO_LARGE: return "problem exceeds the built-in scratch (GRAWA_STATIC_MAX_PARTIALS)";
    }
    return "unknown status";
}

const char* grawa_last_cuda_error(void) { return t_cuda_error.c_str(); }

size_t grawa_workspace_bytes(int64_t n, int M, const int64_t* layer_offsets, int n_layers)
{
    if (M < 1 || M > GRAWA_MAX_WORKERS || n < 0 || n_layers < 0 || (layer_offsets == nullptr) != (n_layers == 0)) return 0;
    std::vector<int64_t> off;
    if (layer_offsets) {
        if (layer_offsets[0] != 0 || layer_offsets[n_layers] != n) return 0;
        for (int k = 0; k < n_layers; ++k)
            if (layer_offsets[k + 1] < layer_offsets[k]) return 0;
        off.assign(layer_offsets, layer_offsets + n_layers + 1);
    } else {
        off.assign({0, n});
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    return workspace_layout(static_cast<int>(off.size()) - 1, M).total;
}

grawa_status grawa_mgrawa_step(float* const* params, const float* const* grads, int64_t n, int M, float pull,
                               const int64_t* layer_offsets, int n_layers, float* center_out,
                               const grawa_options* options, grawa_stream_t stream)
{
    return step_entry(kMgrawa, params, grads, GivenScores{}, n, M, pull, layer_offsets, n_layers, center_out, options, stream);
}

grawa_status grawa_grawa_step(float* const* params, const float* const* grads, int64_t n, int M, float pull,
                              const int64_t* layer_offsets, int n_layers, float* center_out,
                              const grawa_options* options, grawa_stream_t stream)
{
    return step_entry(kGrawa, params, grads, GivenScores{}, n, M, pull, layer_offsets, n_layers, center_out, options, stream);
}

grawa_status grawa_lgrawa_step(float* const* params, const float* const* grads, int64_t n, int M, float pull,
                               const int64_t* layer_offsets, int n_layers, float* center_out,
                               const grawa_options* options, grawa_stream_t stream)
{
    return step_entry(kLgrawa, params, grads, GivenScores{}, n, M, pull, layer_offsets, n_layers, center_out, options, stream);
}

grawa_status grawa_step_typed(grawa_dtype dtype, grawa_variant variant, void* const* params, const void* const* grads, int64_t n,
                              int M, float pull, const int64_t* layer_offsets, int n_layers, void* center_out,
                              const grawa_options* options, grawa_stream_t stream)
{
    if (variant != GRAWA_VARIANT_GRAWA && variant != GRAWA_VARIANT_MGRAWA && variant != GRAWA_VARIANT_LGRAWA)
        return GRAWA_ERR_INVALID_ARG;
    if (dtype != GRAWA_F32 && dtype != GRAWA_BF16 && dtype != GRAWA_F16) return GRAWA_ERR_INVALID_ARG;
    // the pointer tables carry untyped addresses; the kernels of `dtype` give them their element type
    return step_entry(static_cast<int>(variant), reinterpret_cast<float* const*>(params),
                      reinterpret_cast<const float* const*>(grads), GivenScores{}, n, M, pull, layer_offsets, n_layers,
                      static_cast<float*>(center_out), options, stream, static_cast<int>(dtype));
}

grawa_status grawa_step_from_layer_norms_typed(grawa_dtype dtype, grawa_variant variant, void* const* params,
                                               const double* layer_norms, int64_t n, int M, float pull,
                                               const int64_t* layer_offsets, int n_layers, void* center_out,
                                               const grawa_options* options, grawa_stream_t stream)
{
    if (!variant_ok(variant) || !dtype_ok(dtype)) return GRAWA_ERR_INVALID_ARG;
    GivenScores given;
    given.data = layer_norms;
    return step_entry(static_cast<int>(variant), reinterpret_cast<float* const*>(params), nullptr, given, n, M, pull, layer_offsets,
                      n_layers, static_cast<float*>(center_out), options, stream, static_cast<int>(dtype));
}

grawa_status grawa_step_from_layer_norms(grawa_variant variant, float* const* params, const double* layer_norms, int64_t n,
                                         int M, float pull, const int64_t* layer_offsets, int n_layers, float* center_out,
                                         const grawa_options* options, grawa_stream_t stream)
{
    return grawa_step_from_layer_norms_typed(GRAWA_F32, variant, reinterpret_cast<void* const*>(params), layer_norms, n, M, pull,
                                             layer_offsets, n_layers, center_out, options, stream);
}

grawa_status grawa_step_from_layer_sums_typed(grawa_dtype dtype, grawa_variant variant, void* const* params,
                                              const double* layer_sums, int parts, int64_t n, int M, float pull,
                                              const int64_t* layer_offsets, int n_layers, void* center_out,
                                              const grawa_options* options, grawa_stream_t stream)
{
    if (!variant_ok(variant) || !dtype_ok(dtype)) return GRAWA_ERR_INVALID_ARG;
    GivenScores given;
    given.data = layer_sums; given.parts = parts; given.sums = 1;
    return step_entry(static_cast<int>(variant), reinterpret_cast<float* const*>(params), nullptr, given, n, M, pull, layer_offsets,
                      n_layers, static_cast<float*>(center_out), options, stream, static_cast<int>(dtype));
}

grawa_status grawa_step_from_layer_sums(grawa_variant variant, float* const* params, const double* layer_sums, int parts,
                                        int64_t n, int M, float pull, const int64_t* layer_offsets, int n_layers,
                                        float* center_out, const grawa_options* options, grawa_stream_t stream)
{
    return grawa_step_from_layer_sums_typed(GRAWA_F32, variant, reinterpret_cast<void* const*>(params), layer_sums, parts, n, M,
                                            pull, layer_offsets, n_layers, center_out, options, stream);
}

grawa_status grawa_layer_sumsq_typed(grawa_dtype dtype, const void* const* grads, int64_t n, int M,
                                     const int64_t* layer_offsets, int n_layers, double* sumsq_out, grawa_stream_t stream)
{
    if (grads == nullptr || sumsq_out == nullptr || M < 1 || M > GRAWA_MAX_WORKERS || !dtype_ok(dtype)) return GRAWA_ERR_INVALID_ARG;
    // validate() wants parameter vectors; the gradients stand in (nothing is written through them)
    std::vector<float*> fake(M);
    for (int m = 0; m < M; ++m) fake[m] = static_cast<float*>(const_cast<void*>(grads[m]));
    std::vector<int64_t> off;
    grawa_status st = validate(fake.data(), nullptr, n, M, 0.0f, layer_offsets, n_layers, nullptr, &off, elem_size(dtype));
    if (st != GRAWA_OK) return st;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (n == 0) {                                    // nothing to add up: every sum is zero
        GRAWA_CUDA_TRY(cudaMemsetAsync(sumsq_out, 0, sizeof(double) * (off.size() - 1) * M, stream));
        return GRAWA_OK;
    }
    Plan* plan = nullptr;
    st = get_plan(n, M, off, stream, &plan, dtype == GRAWA_F32 ? 4 : 2);
    if (st != GRAWA_OK) return st;
    grawa_options opt{};
    opt.sumsq_out = sumsq_out;
    StepContext c;
    st = make_context(kLgrawa, fake.data(), reinterpret_cast<const float* const*>(grads), n, M, 0.0f, nullptr, &opt, stream, plan, &c);
    if (st != GRAWA_OK) return st;
    c.dtype = static_cast<int>(dtype);
    return enqueue_weights(c);
}

grawa_status grawa_layer_sumsq(const float* const* grads, int64_t n, int M, const int64_t* layer_offsets, int n_layers,
                               double* sumsq_out, grawa_stream_t stream)
{
    return grawa_layer_sumsq_typed(GRAWA_F32, reinterpret_cast<const void* const*>(grads), n, M, layer_offsets, n_layers, sumsq_out,
                                   stream);
}

grawa_status grawa_layer_norms_typed(grawa_dtype dtype, const void* grad, int64_t n, const int64_t* layer_offsets, int n_layers,
                                     double* norms_out, grawa_stream_t stream)
{
    if (grad == nullptr || norms_out == nullptr || n < 0 || !dtype_ok(dtype)) return GRAWA_ERR_INVALID_ARG;
    // validate() wants a parameter vector; the gradient stands in (nothing is written through it)
    float* fake_params[1] = {static_cast<float*>(const_cast<void*>(grad))};
    std::vector<int64_t> off;
    grawa_status st = validate(fake_params, nullptr, n, 1, 0.0f, layer_offsets, n_layers, nullptr, &off, elem_size(dtype));
    if (st != GRAWA_OK || n == 0) return st;
    std::lock_guard<std::mutex> lock(g_mutex);
    Plan* plan = nullptr;
    st = get_plan(n, 1, off, stream, &plan, dtype == GRAWA_F32 ? 4 : 2);
    if (st != GRAWA_OK) return st;
    grawa_options opt{};
    opt.scores_out = norms_out;
    const float* grads[1] = {static_cast<const float*>(grad)};
    StepContext c;
    st = make_context(kLgrawa, fake_params, grads, n, 1, 0.0f, nullptr, &opt, stream, plan, &c);
    if (st != GRAWA_OK) return st;
    c.dtype = static_cast<int>(dtype);
    return enqueue_weights(c);
}

grawa_status grawa_layer_norms(const float* grad, int64_t n, const int64_t* layer_offsets, int n_layers, double* norms_out,
                               grawa_stream_t stream)
{
    return grawa_layer_norms_typed(GRAWA_F32, grad, n, layer_offsets, n_layers, norms_out, stream);
}

grawa_status grawa_norm_ema(double* g_mvg, const double* g_cur, int n_layers, double gamma, int64_t t, double* g_est,
                            grawa_stream_t stream)
{
    if (g_mvg == nullptr || g_cur == nullptr || g_est == nullptr || n_layers < 0 || t < 1) return GRAWA_ERR_INVALID_ARG;
    if (!(gamma >= 0.0 && gamma < 1.0)) return GRAWA_ERR_INVALID_ARG;
    if (n_layers == 0) return GRAWA_OK;
    const double corr = 1.0 - std::pow(gamma, static_cast<double>(t));
    GRAWA_CUDA_TRY(launch_kernel(norm_ema_kernel, (n_layers + kThreads - 1) / kThreads, kThreads, stream, false, g_mvg, g_cur,
                                 n_layers, gamma, corr, g_est));
    return GRAWA_OK;
}

grawa_status grawa_step_host_typed(grawa_dtype dtype, grawa_variant variant, void* const* params, const void* const* grads,
                                   int64_t n, int M, float pull, const int64_t* layer_offsets, int n_layers, void* center_out,
                                   grawa_stream_t stream)
{
    if (!variant_ok(variant) || !dtype_ok(dtype) || grads == nullptr) return GRAWA_ERR_INVALID_ARG;
    const size_t es = elem_size(dtype);
    std::vector<int64_t> off;
    grawa_status st = validate(reinterpret_cast<float* const*>(params), reinterpret_cast<const float* const*>(grads), n, M, pull,
                               layer_offsets, n_layers, static_cast<const float*>(center_out), &off, es);
    if (st != GRAWA_OK || n == 0) return st;
    std::lock_guard<std::mutex> lock(g_mutex);
    Plan* plan = nullptr;
    st = get_plan(n, M, off, stream, &plan, dtype == GRAWA_F32 ? 4 : 2);
    if (st != GRAWA_OK) return st;
    const size_t nn = align_up(static_cast<size_t>(n), 128);     // keeps every staged vector 256-byte aligned
    if (!plan->d_stage) GRAWA_CUDA_TRY(cudaMalloc(&plan->d_stage, es * nn * (2 * static_cast<size_t>(M) + 1)));
    if (!plan->d2h_stream) GRAWA_CUDA_TRY(cudaStreamCreateWithFlags(&plan->d2h_stream, cudaStreamNonBlocking));
    char* stage = reinterpret_cast<char*>(plan->d_stage);
    std::vector<float*> dx(M);                        // untyped device addresses; the kernels of `dtype` type them
    std::vector<const float*> dg(M);
    char* dc = stage + es * nn * 2 * M;
    const size_t bytes = es * static_cast<size_t>(n);
    for (int m = 0; m < M; ++m) {
        dg[m] = reinterpret_cast<const float*>(stage + es * nn * m);
        dx[m] = reinterpret_cast<float*>(stage + es * nn * (M + m));
        GRAWA_CUDA_TRY(cudaMemcpyAsync(stage + es * nn * m, grads[m], bytes, cudaMemcpyHostToDevice, stream));
    }
    StepContext c;
    st = make_context(variant, dx.data(), dg.data(), n, M, pull, center_out ? reinterpret_cast<float*>(dc) : nullptr, nullptr, stream,
                      plan, &c);
    if (st != GRAWA_OK) return st;
    c.dtype = static_cast<int>(dtype);
    st = enqueue_weights(c);                          // runs while the parameters are still arriving
    if (st != GRAWA_OK) return st;
    if (M == 1) {
        // identity: the worker is untouched; the centre is the worker itself
        if (center_out) std::memcpy(center_out, params[0], bytes);
        GRAWA_CUDA_TRY(cudaStreamSynchronize(stream));
        return GRAWA_OK;
    }
    // Centre+pull in chunks of work items: upload the chunk of all M workers, run it, and download
    // its results on a second stream while the next chunk is being uploaded (the two directions of
    // the host link work at the same time).
    const bool per_layer = static_cast<int>(variant) == kLgrawa;
    const int items = c.pull_items;
    const int64_t chunk_elems = std::max<int64_t>(int64_t{1} << 20, (n + 15) / 16);
    auto item_begin_elem = [&](int i) -> int64_t {
        if (i >= items) return n;
        return per_layer ? plan->h_segs2[i].begin : static_cast<int64_t>(i) * plan->tile2;
    };
    size_t ev_used = 0;
    int i0 = 0;
    while (i0 < items) {
        int i1 = i0 + 1;
        const int64_t e0 = item_begin_elem(i0);
        while (i1 < items && item_begin_elem(i1) - e0 < chunk_elems) ++i1;
        const int64_t e1 = item_begin_elem(i1);
        const size_t cb = es * static_cast<size_t>(e1 - e0), o0 = es * static_cast<size_t>(e0);
        for (int m = 0; m < M; ++m)
            GRAWA_CUDA_TRY(cudaMemcpyAsync(reinterpret_cast<char*>(dx[m]) + o0, static_cast<const char*>(params[m]) + o0, cb,
                                           cudaMemcpyHostToDevice, stream));
        if (plan->bulk) GRAWA_CUDA_TRY(cudaMemsetAsync(c.counter, 0, sizeof(unsigned), stream));
        st = enqueue_center_pull(c, i0, i1);
        if (st != GRAWA_OK) return st;
        if (ev_used == plan->events.size()) {
            cudaEvent_t ev;
            GRAWA_CUDA_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
            plan->events.push_back(ev);
        }
        cudaEvent_t ev = plan->events[ev_used++];
        GRAWA_CUDA_TRY(cudaEventRecord(ev, stream));
        GRAWA_CUDA_TRY(cudaStreamWaitEvent(plan->d2h_stream, ev, 0));
        for (int m = 0; m < M; ++m)
            GRAWA_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(params[m]) + o0, reinterpret_cast<char*>(dx[m]) + o0, cb,
                                           cudaMemcpyDeviceToHost, plan->d2h_stream));
        if (center_out)
            GRAWA_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(center_out) + o0, dc + o0, cb, cudaMemcpyDeviceToHost, plan->d2h_stream));
        i0 = i1;
    }
    GRAWA_CUDA_TRY(cudaStreamSynchronize(plan->d2h_stream));
    GRAWA_CUDA_TRY(cudaStreamSynchronize(stream));
    return GRAWA_OK;
}

grawa_status grawa_step_host(grawa_variant variant, float* const* params, const float* const* grads, int64_t n, int M,
                             float pull, const int64_t* layer_offsets, int n_layers, float* center_out,
                             grawa_stream_t stream)
{
    return grawa_step_host_typed(GRAWA_F32, variant, reinterpret_cast<void* const*>(params),
                                 reinterpret_cast<const void* const*>(grads), n, M, pull, layer_offsets, n_layers, center_out, stream);
}

grawa_status grawa_last_step_status(grawa_stream_t stream)
{
    int device = 0;
    GRAWA_CUDA_TRY(cudaGetDevice(&device));
    int* status = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        auto it = g_last_status.find({device, stream});
        if (it == g_last_status.end()) return GRAWA_ERR_INVALID_ARG;
        status = it->second;
    }
    GRAWA_CUDA_TRY(cudaStreamSynchronize(stream));
    int word = 0;
    GRAWA_CUDA_TRY(cudaMemcpy(&word, status, sizeof word, cudaMemcpyDeviceToHost));
    if (word & kStatusTimeout) return GRAWA_ERR_TIMEOUT;
    if (word & kStatusNonFinite) return GRAWA_ERR_NONFINITE;
    return GRAWA_OK;
}

grawa_status grawa_prox_step_typed(grawa_dtype dtype, void* const* params, const void* center, int64_t n, int M,
                                   float mu_over_tau, grawa_stream_t stream)
{
    if (!dtype_ok(dtype) || (center == nullptr && n > 0)) return GRAWA_ERR_INVALID_ARG;
    std::vector<int64_t> off;
    grawa_status st = validate(reinterpret_cast<float* const*>(params), nullptr, n, M, mu_over_tau, nullptr, 0,
                               static_cast<const float*>(center), &off, elem_size(dtype));
    if (st != GRAWA_OK || n == 0) return st;
    MutPtrs xp{};
    bool vec = aligned16(center), wide = (reinterpret_cast<uintptr_t>(center) & 31u) == 0;
    for (int m = 0; m < M; ++m) {
        xp.p[m] = static_cast<float*>(params[m]);
        vec = vec && aligned16(params[m]);
        wide = wide && (reinterpret_cast<uintptr_t>(params[m]) & 31u) == 0;
    }
    int64_t tile;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        wide = wide && g_pull_wide && dtype == GRAWA_F32;     // (on 16-bit storage 32-byte columns measured no gain)
        // one vector column per thread (measured best): 16 bytes, or for fp32 32 bytes when every base is 32-byte aligned
        tile = g_pull_tile > 0 ? g_pull_tile : (wide ? 32 : 16) * kThreads / static_cast<int64_t>(elem_size(dtype));
    }
    const int64_t tiles = (n + tile - 1) / tile;
    if (tiles > 0x7fffffffll) return GRAWA_ERR_INVALID_ARG;
    const int grid = static_cast<int>(tiles), t = static_cast<int>(tile), v = vec ? 1 : 0;
    if (dtype == GRAWA_BF16)
        prox16_kernel<__nv_bfloat16><<<grid, kThreads, 0, stream>>>(xp, static_cast<const __nv_bfloat16*>(center), n, t, mu_over_tau, M, v);
    else if (dtype == GRAWA_F16)
        prox16_kernel<__half><<<grid, kThreads, 0, stream>>>(xp, static_cast<const __half*>(center), n, t, mu_over_tau, M, v);
    else
        (wide ? prox_kernel<8> : prox_kernel<4>)<<<grid, kThreads, 0, stream>>>(xp, static_cast<const float*>(center), n, t, mu_over_tau, M, v);
    ++g_launches;
    GRAWA_CUDA_TRY(cudaGetLastError());
    return GRAWA_OK;
}

grawa_status grawa_prox_step(float* const* params, const float* center, int64_t n, int M, float mu_over_tau,
                             grawa_stream_t stream)
{
    return grawa_prox_step_typed(GRAWA_F32, reinterpret_cast<void* const*>(params), center, n, M, mu_over_tau, stream);
}

grawa_status grawa_sumsq_static(const float* const* grads, int64_t n, int M, double* sumsq_out, grawa_stream_t stream)
{
    if (grads == nullptr || sumsq_out == nullptr || M < 1 || M > GRAWA_MAX_WORKERS || n < 0) return GRAWA_ERR_INVALID_ARG;
    ConstPtrs gp{};
    bool vec = true;
    for (int m = 0; m < M; ++m) {
        if (n > 0 && (grads[m] == nullptr || (reinterpret_cast<uintptr_t>(grads[m]) & 3u))) return GRAWA_ERR_INVALID_ARG;
        gp.p[m] = grads[m];
        vec = vec && aligned16(grads[m]);
    }
    const int64_t tiles64 = (n + kStaticTile - 1) / kStaticTile;
    if (tiles64 * M > GRAWA_STATIC_MAX_PARTIALS) return GRAWA_ERR_TOO_LARGE;
    const int tiles = static_cast<int>(tiles64);

    // Once per device, with that device current: the device address of the built-in array.
    int device = 0;
    GRAWA_CUDA_TRY(cudaGetDevice(&device));
    if (device < 0 || device >= kMaxDevices) return GRAWA_ERR_INVALID_ARG;
    double* partials = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (g_static_partials_addr[device] == nullptr) {
            double* addr = nullptr;
            GRAWA_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&addr), g_static_partials));
            g_static_partials_addr[device] = addr;
        }
        partials = g_static_partials_addr[device];
    }
    if (tiles > 0) {
        sumsq_flat_kernel<8><<<tiles * M, kThreads, 0, stream>>>(gp, n, tiles, kStaticTile, partials, vec ? 1 : 0);
        ++g_launches;
        GRAWA_CUDA_TRY(cudaGetLastError());
    }
    // with tiles == 0 every row is empty and the sums are written as zeros
    sum_partials_kernel<<<M, kFinalizeThreads, 0, stream>>>(partials, tiles, sumsq_out);
    ++g_launches;
    GRAWA_CUDA_TRY(cudaGetLastError());
    return GRAWA_OK;
}

grawa_status grawa_selftest_bounded_wait(int64_t limit_ns, grawa_stream_t stream)
{
    if (limit_ns < 1000 || limit_ns > 1000000000) return GRAWA_ERR_INVALID_ARG;
    int device = 0;
    GRAWA_CUDA_TRY(cudaGetDevice(&device));
    if (device < 0 || device >= kMaxDevices) return GRAWA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    static int* words[kMaxDevices] = {};
    if (words[device] == nullptr) GRAWA_CUDA_TRY(cudaMalloc(&words[device], sizeof(int)));
    GRAWA_CUDA_TRY(cudaMemsetAsync(words[device], 0, sizeof(int), stream));
    g_last_status[{device, stream}] = words[device];
    GRAWA_CUDA_TRY(launch_kernel(bounded_wait_selftest_kernel, 1, kThreads, stream, false, words[device],
                                 static_cast<unsigned long long>(limit_ns)));
    return GRAWA_OK;
}

int64_t grawa_debug_bounds_violations(int selfcheck)
{
#ifdef GRAWA_DEBUG_BOUNDS
    if (selfcheck) bounds_selfcheck_kernel<<<1, 32>>>();
    if (cudaDeviceSynchronize() != cudaSuccess) return -2;
    int count = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&count, g_bounds_violations, sizeof count) != cudaSuccess) return -2;
    if (cudaMemcpyToSymbol(g_bounds_violations, &zero, sizeof zero) != cudaSuccess) return -2;
    return count;
#else
    (void)selfcheck;
    return -1;
#endif
}

int grawa_trace_read(uint64_t* rows_out, int max_rows)
{
#ifdef GRAWA_TRACE
    if (cudaDeviceSynchronize() != cudaSuccess) return -2;
    static TraceRow host[kTraceRows][kTraceKinds];
    unsigned arrivals[kTraceKinds] = {};
    if (rows_out != nullptr && max_rows > 0) {
        if (cudaMemcpyFromSymbol(host, g_trace, sizeof host) != cudaSuccess) return -2;
        const int rows = std::min(max_rows, kTraceRows);
        std::memcpy(rows_out, host, sizeof(TraceRow) * kTraceKinds * static_cast<size_t>(rows));
    }
    for (auto& row : host)
        for (auto& r : row) r = TraceRow{~0ull, ~0ull, 0ull, 0ull};
    if (cudaMemcpyToSymbol(g_trace, host, sizeof host) != cudaSuccess) return -2;
    if (cudaMemcpyToSymbol(g_trace_arrivals, arrivals, sizeof arrivals) != cudaSuccess) return -2;
    return kTraceRows;
#else
    (void)rows_out; (void)max_rows;
    return -1;
#endif
}

static void clear_plans_locked()
{
    cudaDeviceSynchronize();
    g_recent_plan = nullptr;
    g_plans.clear();
    g_last_status.clear();
}

grawa_status grawa_set_option(const char* name, int64_t value)
{
    if (name == nullptr) return GRAWA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    const bool tile_ok = value >= 1024 && value <= 1048576 && value % 1024 == 0;
    if (std::strcmp(name, "sumsq_tile") == 0) {
        if (!tile_ok) return GRAWA_ERR_INVALID_ARG;
        if (value != g_sumsq_tile) { g_sumsq_tile = value; clear_plans_locked(); }
        return GRAWA_OK;
    }
    if (std::strcmp(name, "pull_tile") == 0) {
        if (!tile_ok && value != 0) return GRAWA_ERR_INVALID_ARG;
        if (value != g_pull_tile) { g_pull_tile = value; clear_plans_locked(); }
        return GRAWA_OK;
    }
    if (std::strcmp(name, "pull_variant") == 0) {
        if (value < 0 || value > 2) return GRAWA_ERR_INVALID_ARG;
        if (value != g_pull_variant) { g_pull_variant = value; clear_plans_locked(); }
        return GRAWA_OK;
    }
    if (std::strcmp(name, "bulk_tile") == 0) {
        if (value < 0 || value > 16384 || value % 256 != 0) return GRAWA_ERR_INVALID_ARG;
        if (value != g_bulk_tile) { g_bulk_tile = value; clear_plans_locked(); }
        return GRAWA_OK;
    }
    if (std::strcmp(name, "kernel_timing") == 0) {
        if (value < 0 || value > 1) return GRAWA_ERR_INVALID_ARG;
        g_kernel_timing = value;
        return GRAWA_OK;
    }
    if (std::strcmp(name, "dependent_launch") == 0) {
        if (value < 0 || value > 1) return GRAWA_ERR_INVALID_ARG;
        g_pdl = value;
        return GRAWA_OK;
    }
    if (std::strcmp(name, "pull_prefetch_waves") == 0 || std::strcmp(name, "sumsq_prefetch_waves") == 0) {
        if (value < 0 || value > 8) return GRAWA_ERR_INVALID_ARG;
        (name[0] == 'p' ? g_pull_prefetch_waves : g_sumsq_prefetch_waves) = value;
        return GRAWA_OK;
    }
    if (std::strcmp(name, "pull_preload") == 0) {
        if (value < 0 || value > 1) return GRAWA_ERR_INVALID_ARG;
        g_pull_preload = value;
        return GRAWA_OK;
    }
    if (std::strcmp(name, "pull_wide") == 0) {
        if (value < 0 || value > 1) return GRAWA_ERR_INVALID_ARG;
        g_pull_wide = value;
        return GRAWA_OK;
    }
    if (std::strcmp(name, "pull16_staged") == 0) {
        if (value < 0 || value > 1) return GRAWA_ERR_INVALID_ARG;
        if (value != g_pull16_staged) { g_pull16_staged = value; clear_plans_locked(); }
        return GRAWA_OK;
    }
    if (std::strcmp(name, "sumsq_ctas_per_sm") == 0 || std::strcmp(name, "pull_ctas_per_sm") == 0) {
        if (value < 0 || value > 32) return GRAWA_ERR_INVALID_ARG;
        (name[0] == 's' ? g_sumsq_ctas_per_sm : g_pull_ctas_per_sm) = value;
        return GRAWA_OK;
    }
    return GRAWA_ERR_INVALID_ARG;
}

int64_t grawa_get_option(const char* name)
{
    if (name == nullptr) return -1;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (std::strcmp(name, "sumsq_tile") == 0) return g_sumsq_tile;
    if (std::strcmp(name, "pull_tile") == 0) return g_pull_tile;
    if (std::strcmp(name, "pull_variant") == 0) return g_pull_variant;
    if (std::strcmp(name, "bulk_tile") == 0) return g_bulk_tile;
    if (std::strcmp(name, "kernel_timing") == 0) return g_kernel_timing;
    if (std::strcmp(name, "dependent_launch") == 0) return g_pdl;
    if (std::strcmp(name, "pull_preload") == 0) return g_pull_preload;
    if (std::strcmp(name, "pull_wide") == 0) return g_pull_wide;
    if (std::strcmp(name, "pull16_staged") == 0) return g_pull16_staged;
    if (std::strcmp(name, "pull_prefetch_waves") == 0) return g_pull_prefetch_waves;
    if (std::strcmp(name, "sumsq_prefetch_waves") == 0) return g_sumsq_prefetch_waves;
    if (std::strcmp(name, "sumsq_ctas_per_sm") == 0) return g_sumsq_ctas_per_sm;
    if (std::strcmp(name, "pull_ctas_per_sm") == 0) return g_pull_ctas_per_sm;
    return -1;
}

int64_t grawa_launch_count(void) { return g_launches.load(); }

grawa_status grawa_collect_kernel_times(double* sumsq_ms, double* finalize_ms, double* center_pull_ms, int64_t* steps)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    GRAWA_CUDA_TRY(cudaDeviceSynchronize());
    double sum[3] = {0.0, 0.0, 0.0};
    for (size_t i = 0; i < g_timed_used; ++i)
        for (int ph = 0; ph < 3; ++ph) {
            float ms = 0.f;
            GRAWA_CUDA_TRY(cudaEventElapsedTime(&ms, g_timed_pool[i].e[ph], g_timed_pool[i].e[ph + 1]));
            sum[ph] += ms;
        }
    if (sumsq_ms) *sumsq_ms = sum[0];
    if (finalize_ms) *finalize_ms = sum[1];
    if (center_pull_ms) *center_pull_ms = sum[2];
    if (steps) *steps = static_cast<int64_t>(g_timed_used);
    g_timed_used = 0;
    return GRAWA_OK;
}

void grawa_clear_plans(void)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    clear_plans_locked();
}

}  // extern "C"
