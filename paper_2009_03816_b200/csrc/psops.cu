// psops.cu -- C ABI and host side of the PSO-PS synchronisation stage (kernels: psops_kernels.cuh).
//
// The paper's synchronisation stage (Algorithm 1, sync branch; Algorithm 3;
// Eq. 5-7) over K particles stored as K flat fp32 rows in HBM.  The stage is a
// pure streaming pass: per particle-element it reads w, v and (unless the
// particle improved) pBest, and writes v, w and (if it improved) pBest -- five
// 4-byte accesses -- plus one read of the gBest row.  Nothing is a dense
// contraction, so the kernels are bandwidth kernels: 128-bit coalesced
// accesses, one thread owning a 4-element quad for ALL particles (which also
// makes the in-place read of the gBest row safe: the thread that overwrites
// w_g[d] is the one that read gBest[d] first), and the Philox arithmetic
// scheduled into the shadow of the loads.
//
// Floating point: every operation is an explicit round-to-nearest intrinsic;
// the file is compiled with -fmad=false and without fast-math, subnormals
// kept, so the rounding sequence is the one documented in psops.h.

#include "psops.h"

#include <cooperative_groups.h>   // thread-block clusters of the fitness finaliser
#include <cuda_runtime.h>

#include <cmath>
#include <cstddef>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "psops_kernels.cuh"

// Bytes of weights per pipeline stage of psops_sync_host (all K rows of one
// element range): large enough for full PCIe efficiency, small enough that
// filling and draining the three-stage pipeline stays a small share.
#ifndef PSOPS_HOST_CHUNK_BYTES
#define PSOPS_HOST_CHUNK_BYTES (64ll << 20)
#endif

// Share of the L2 cache that the arrays kept resident (write-back accesses
// instead of evict-first ones) may take up together.  Measured on B200 (126 MB
// of L2, K = 8, time per sync from a CUDA graph, arrays of 4 K N bytes each):
//   array   all streamed   x resident   x, v resident   all resident
//   19 MB      13.6 us        13.3          13.2            13.1
//   32 MB      24.3           23.1          22.5            24.9
//   40 MB      33.5           30.5          30.6            34.4
//   64 MB      52.8           46.5          54.2            53.7
//   80 MB      66.8           64.5          69.0            67.8
//  102 MB      82.4           85.0          85.0            83.8
// i.e. keep as many arrays as fit in about half of L2.
#ifndef PSOPS_L2_RESIDENT_PERCENT
#define PSOPS_L2_RESIDENT_PERCENT 52
#endif

namespace {

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
    size_t off_losses, off_pbest_loss, off_desc, off_gbest, off_partials, total;
};

bool config_ok(const psops_config *c)
{
    if (c == nullptr) return false;
    if (c->K < 1 || c->K > PSOPS_MAX_K) return false;
    if (c->N < 1 || c->N >= (1ll << 33)) return false;
    if (c->ld < c->N) return false;
    if (c->t_max < 1) return false;
    if (!std::isfinite(c->m_max) || !std::isfinite(c->m_min)) return false;
    if (!std::isfinite(c->c1) || !std::isfinite(c->c2)) return false;
    if (c->flags & ~(PSOPS_KEEP_GBEST | PSOPS_QUADRATIC | PSOPS_GBEST_HISTORY | PSOPS_SEPARATE_SELECT)) return false;
    // particle shard: rows [k_first, k_first + K) of a swarm of K_total particles
    if (c->K_total == 0) {
        if (c->k_first != 0) return false;
    } else {
        if (c->K_total < c->K || c->K_total > PSOPS_MAX_K) return false;
        if (c->k_first < 0 || c->k_first + c->K > c->K_total) return false;
        if (c->K_total > c->K && (c->flags & (PSOPS_QUADRATIC | PSOPS_GBEST_HISTORY))) return false;
    }
    return true;
}

inline int swarm_size(const psops_config *c) { return c->K_total ? c->K_total : c->K; }
inline bool keeps_gbest(const psops_config *c) { return (c->flags & (PSOPS_KEEP_GBEST | PSOPS_GBEST_HISTORY)) != 0; }

// Many particles on few elements: the update splits the rows over blockIdx.y
// (see psops_sync) and then needs a snapshot of the gBest row, N floats of
// workspace.  Whether a swarm may be split depends on its shape only, so that
// the workspace size does not depend on the device.
#ifndef PSOPS_SPLIT_MAX_ELEMENTS
#define PSOPS_SPLIT_MAX_ELEMENTS (1ll << 19)
#endif
constexpr int kSplitMinParticles = 9;           // below: the single-launch form or one group
constexpr int kSplitRowsPerGroup = 4;           // at least this many rows per group (one full batch)
inline bool may_split_rows(const psops_config *c)
{
    return c->K >= kSplitMinParticles && c->N <= PSOPS_SPLIT_MAX_ELEMENTS &&
           !(c->flags & (PSOPS_QUADRATIC | PSOPS_GBEST_HISTORY)) && swarm_size(c) == c->K;
}

Layout make_layout(const psops_config *c)
{
    Layout L{};
    const size_t kbytes = round_up(sizeof(float) * (size_t)swarm_size(c), 256);
    size_t at = 0;
    L.off_losses = at;      at += kbytes;
    L.off_pbest_loss = at;  at += kbytes;
    L.off_desc = at;        at += round_up(sizeof(SyncDesc), 256);
    L.off_gbest = at;
    if (keeps_gbest(c) || may_split_rows(c)) at += round_up(sizeof(float) * (size_t)round_up((size_t)c->N, 4), 256);
    L.off_partials = at;
    if (c->flags & PSOPS_QUADRATIC) {
        const size_t tiles = ((size_t)c->N + kTileElems - 1) / kTileElems;
        at += round_up(sizeof(double) * tiles * (size_t)c->K, 256);
    }
    L.total = at;
    return L;
}

float inertia_of(const psops_config *c, int64_t t)
{
    // Eq. 5 in double from the fp32 hyper-parameters, rounded once.
    if (t < 0) t = 0;
    if (t > c->t_max) t = c->t_max;
    const double m = (double)c->m_max - (double)t * ((double)c->m_max - (double)c->m_min) / (double)c->t_max;
    return (float)m;
}

} // namespace

struct psops_ctx {
    psops_config cfg;
    Layout lay;
    float *x, *v, *p;
    char *ws;
    float *d_losses, *d_pbest_loss, *d_gbest;
    const float *loss_src;             // where the next selection reads the losses: d_losses or the caller's device buffer
    SyncDesc *d_desc;
    double *d_partials;
    const float *dvec, *tvec;
    cudaStream_t stream;
    cudaStream_t s_in, s_out;          // copy streams of psops_sync_host
    std::vector<cudaEvent_t> events;
    int device;
    bool aligned;
    bool have_losses;
    bool synced_once;
    bool selected;                     // psops_shard_select ran and the update of that sync is not complete yet
    long long range_next;              // first element the next psops_shard_update_range must start at
    int *h_g;                          // page-locked, device-mapped word the selection kernel writes g to (shards)
    int *d_g;                          // the same word as the device sees it
    cudaEvent_t ev_select;             // recorded behind the selection kernel of a shard
    int resident_arrays;               // how many of x, v, pbest are accessed write-back (kept in L2); the rest is streamed
    float *d_snapshot;                 // N floats for the gBest snapshot of a row-split update (the kept copy, if one is kept)
    int row_groups;                    // > 1: psops_sync splits the rows into this many groups over blockIdx.y
    int group_rows;                    // rows per group
    long long one_wave_blocks;         // blocks of the select-in-update kernel that are resident at once on this GPU
    int Kt;                            // particles in the whole swarm (= cfg.K unless sharded)
    uint32_t step;                     // syncs enqueued through this context (the stream's own counter is on the device)
    long long quads, tiles;
    int64_t launches;
    char err[256];
};

namespace {

int cuda_fail(psops_ctx *ctx, cudaError_t e, const char *what)
{
    if (ctx) std::snprintf(ctx->err, sizeof(ctx->err), "%s: %s", what, cudaGetErrorString(e));
    return PSOPS_ECUDA;
}

#define PSOPS_CUDA(ctx, call)                                         \
    do {                                                              \
        cudaError_t e_ = (call);                                      \
        if (e_ != cudaSuccess) return cuda_fail((ctx), e_, #call);    \
    } while (0)

int check_launch(psops_ctx *ctx, const char *what)
{
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, what);
    ctx->launches += 1;
    return PSOPS_OK;
}

// Work of a context belongs to the device that was current at psops_create.
// Entry points that touch the device switch to it if the caller has another
// one current, and switch back on return.
class DeviceGuard {
public:
    explicit DeviceGuard(const psops_ctx *ctx) : previous_(-1)
    {
        int now = -1;
        if (ctx != nullptr && cudaGetDevice(&now) == cudaSuccess && now != ctx->device &&
            cudaSetDevice(ctx->device) == cudaSuccess)
            previous_ = now;
    }
    ~DeviceGuard()
    {
        if (previous_ >= 0) cudaSetDevice(previous_);
    }
    DeviceGuard(const DeviceGuard &) = delete;
    DeviceGuard &operator=(const DeviceGuard &) = delete;

private:
    int previous_;
};

void fill_round_keys(uint64_t seed, uint32_t (&rk)[20])
{
    uint32_t k0 = (uint32_t)(seed & 0xffffffffu), k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        rk[2 * r] = k0;
        rk[2 * r + 1] = k1;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
}

int launch_select(psops_ctx *ctx, int *g_mapped = nullptr)
{
    const int threads = (int)round_up((size_t)ctx->Kt, 32);
    psops_select_kernel<<<1, threads, 0, ctx->stream>>>(ctx->loss_src, ctx->d_losses, ctx->d_pbest_loss,
                                                        ctx->d_desc, ctx->Kt,
                                                        (ctx->cfg.flags & PSOPS_GBEST_HISTORY) ? 1 : 0, g_mapped);
    ctx->loss_src = ctx->d_losses;     // the kernel keeps a copy there
    return check_launch(ctx, "psops_select_kernel");
}

constexpr int kUnroll = PSOPS_UPDATE_UNROLL, kQuads = PSOPS_UPDATE_QUADS;
constexpr int kFitUnroll = PSOPS_FITNESS_UNROLL, kFitQuads = PSOPS_FITNESS_QUADS;
static_assert(32 % kUnroll == 0 && 32 % kFitUnroll == 0, "the improved mask is reloaded every 32 particles");
static_assert(kUpdateThreads % 32 == 0, "a warp must cover whole 128-element tiles");

// Launch with programmatic stream serialisation: the grid may become resident
// while the kernel in front of it in the stream is still running; the kernel
// itself waits (griddepcontrol.wait) for that kernel to finish before it reads
// anything.  For a kernel that does not trigger early this is an ordinary launch.
template <typename... Params, typename... Args>
cudaError_t launch_serialized(bool programmatic, void (*kernel)(Params...), dim3 grid, dim3 block,
                              cudaStream_t stream, Args &&...args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = programmatic ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

using UpdateKernel = void (*)(const UpdateParams);

// Particles in flight per thread.  With few rows (K <= kFewParticles) a deep
// batch is mostly empty; one particle at a time needs half the registers, so
// that five blocks instead of three are resident per SM, which is what a short
// per-thread loop needs to keep the memory system busy (measured on B200 with
// 11 M elements: K = 1: 4.1 -> 6.2 TB/s, K = 2: 5.3 -> 6.7, K = 4: 6.3 -> 6.8,
// K = 8: 6.7 -> 6.8; from K = 16 on the two are equal).  A grid of at most one
// wave is bound by latency instead, and there the deep batch stays (its loads
// are all in flight at once): that is also where the selection is folded in.
constexpr int kFewParticles = 8;
constexpr int kUnrollFew = 1;
// The single-launch form (selection folded in) is for launch-bound swarms: at
// most kSelectMaxParticles particles on a grid of at most one wave.  There the
// per-thread loop over particles is a chain of memory latencies, so the batch
// is as deep as the swarm: four particles in flight up to K = 4, eight beyond
// (152 registers, one block per SM, hence a smaller "one wave").  Measured per
// sync from a CUDA graph, N = 61,706: K = 4: 4.4 us; K = 8: 6.8 us (7.9 with
// four in flight, 7.6 as two kernels).  More particles than that on few
// elements are better served by splitting the rows over more blocks (see
// psops_sync).
constexpr int kSelectMaxParticles = 8;
constexpr int kUnrollSelectDeep = 8;
static_assert(32 % kUnrollSelectDeep == 0 && kSelectMaxParticles <= 32, "one improved-mask word, reloaded every 32 particles");

// All instantiations of kernel (b) for one alignment and one cache policy
// (`resident` arrays of x, v, pbest accessed write-back, the rest streamed).
struct UpdateKernelSet {
    UpdateKernel plain, select, select_deep, few, fitness, split;
};

template <bool ALIGNED, int RESIDENT>
constexpr UpdateKernelSet update_kernel_set()
{
    return {psops_update_kernel<ALIGNED, false, false, RESIDENT, kUnroll, kQuads>,
            psops_update_kernel<ALIGNED, false, true, RESIDENT, kUnroll, kQuads>,
            psops_update_kernel<ALIGNED, false, true, RESIDENT, kUnrollSelectDeep, kQuads>,
            psops_update_kernel<ALIGNED, false, false, RESIDENT, kUnrollFew, kQuads>,
            psops_update_kernel<ALIGNED, true, false, RESIDENT, kFitUnroll, kFitQuads>,
            psops_update_kernel<ALIGNED, false, false, RESIDENT, kUnroll, kQuads, true>};
}

UpdateKernel pick_update_kernel(bool aligned, bool fitness, bool select, int resident, bool few, int K,
                                bool split = false)
{
    static const UpdateKernelSet sets[2][4] = {
        {update_kernel_set<false, 0>(), update_kernel_set<false, 1>(), update_kernel_set<false, 2>(),
         update_kernel_set<false, 3>()},
        {update_kernel_set<true, 0>(), update_kernel_set<true, 1>(), update_kernel_set<true, 2>(),
         update_kernel_set<true, 3>()},
    };
    if (resident < 0 || resident > 3 || (fitness && select)) return nullptr;
    const UpdateKernelSet &set = sets[aligned ? 1 : 0][resident];
    if (split) return (fitness || select) ? nullptr : set.split;
    if (fitness) return set.fitness;
    if (select) return K > kUnroll ? set.select_deep : set.select;
    return few ? set.few : set.plain;
}

// One launch of kernel (b) over quads [q_begin, q_end).  `select`: the launch
// also does the selection of this sync (whole range, K <= 32, see the kernel).
int launch_update(psops_ctx *ctx, float m, float k1, float k2, long long q_begin,
                  long long q_end, bool fitness, cudaStream_t stream, bool programmatic = false,
                  bool select = false, const float *gbest_ext = nullptr, bool split_rows = false)
{
    if (q_end <= q_begin) return PSOPS_OK;
    UpdateParams P{};
    P.x = ctx->x; P.v = ctx->v; P.p = ctx->p;
    P.gbest_copy = ctx->d_gbest;
    P.gbest_ext = gbest_ext;
    P.i_first = ctx->cfg.k_first;
    P.dvec = ctx->dvec; P.tvec = ctx->tvec; P.partials = ctx->d_partials;
    P.desc = ctx->d_desc;
    P.loss_src = ctx->loss_src; P.loss_keep = ctx->d_losses; P.pbest_loss = ctx->d_pbest_loss;
    P.desc_pub = ctx->d_desc;
    P.ld = ctx->cfg.ld; P.N = ctx->cfg.N;
    P.q_begin = q_begin; P.q_end = q_end;
    P.tiles = ctx->tiles;
    P.K = ctx->cfg.K;
    P.group_rows = split_rows ? ctx->group_rows : ctx->cfg.K;
    if (split_rows) P.gbest_copy = nullptr;         // gbest_ext is the snapshot, which is also the kept copy
    P.m = m; P.k1 = k1; P.k2 = k2;
    fill_round_keys(ctx->cfg.seed, P.rk);
    const long long span = q_end - q_begin;
    const int per_block = kUpdateThreads * (fitness ? kFitQuads : kQuads);
    const unsigned blocks = (unsigned)((span + per_block - 1) / per_block);
    const bool few = ctx->cfg.K <= kFewParticles && (long long)blocks > ctx->one_wave_blocks;
    const unsigned groups = split_rows ? (unsigned)ctx->row_groups : 1u;
    const UpdateKernel kernel = pick_update_kernel(ctx->aligned, fitness, select, ctx->resident_arrays, few, ctx->cfg.K,
                                                   split_rows);
    if (kernel == nullptr) return PSOPS_EINVAL;
    const cudaError_t e = launch_serialized(programmatic, kernel, dim3(blocks, groups, 1), dim3(kUpdateThreads, 1, 1), stream, P);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "psops_update_kernel launch");
    if (select) ctx->loss_src = ctx->d_losses;      // the launch keeps a copy there
    return check_launch(ctx, "psops_update_kernel");
}

int launch_finalize(psops_ctx *ctx)
{
    // behind the kernel that writes the tile sums; the finaliser waits for it on the device
    const cudaError_t e = launch_serialized(true, psops_fitness_finalize_kernel, dim3(kFinalizeCluster, ctx->cfg.K),
                                            dim3(kFinalizeCtaThreads, 1, 1), ctx->stream,
                                            (const double *)ctx->d_partials, ctx->d_losses, ctx->tiles);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "psops_fitness_finalize_kernel launch");
    ctx->loss_src = ctx->d_losses;
    return check_launch(ctx, "psops_fitness_finalize_kernel");
}

int validate_sync_args(psops_ctx *ctx, int64_t t_iter, float lambda)
{
    if (ctx == nullptr) return PSOPS_EINVAL;
    if (t_iter < 0) return PSOPS_EINVAL;
    if (!std::isfinite(lambda) || lambda < 1.0f) return PSOPS_EINVAL;
    return PSOPS_OK;
}

int check_host_losses(const float *losses, int K)
{
    if (losses == nullptr) return PSOPS_EINVAL;
    for (int i = 0; i < K; ++i)
        if (losses[i] != losses[i]) return PSOPS_ENAN;
    return PSOPS_OK;
}

// Copy `rows` row pieces of `width` floats between strided buffers.
int copy_rows(psops_ctx *ctx, float *dst, size_t dst_ld, const float *src, size_t src_ld,
              size_t width, int rows, cudaMemcpyKind kind, cudaStream_t stream)
{
    const size_t limit = (size_t)1 << 30;      // stay below the 2-D copy pitch limit
    if (dst_ld * sizeof(float) < limit && src_ld * sizeof(float) < limit) {
        PSOPS_CUDA(ctx, cudaMemcpy2DAsync(dst, dst_ld * sizeof(float), src, src_ld * sizeof(float),
                                          width * sizeof(float), (size_t)rows, kind, stream));
    } else {
        for (int r = 0; r < rows; ++r)
            PSOPS_CUDA(ctx, cudaMemcpyAsync(dst + (size_t)r * dst_ld, src + (size_t)r * src_ld,
                                            width * sizeof(float), kind, stream));
    }
    return PSOPS_OK;
}

int get_event(psops_ctx *ctx, size_t idx, cudaEvent_t *ev)
{
    while (ctx->events.size() <= idx) {
        cudaEvent_t e;
        PSOPS_CUDA(ctx, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        ctx->events.push_back(e);
    }
    *ev = ctx->events[idx];
    return PSOPS_OK;
}

} // namespace

// ---------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------
extern "C" {

size_t psops_workspace_bytes(const psops_config *cfg)
{
    if (!config_ok(cfg)) return 0;
    return make_layout(cfg).total;
}

float psops_inertia(const psops_config *cfg, int64_t t_iter)
{
    if (cfg == nullptr || cfg->t_max < 1) return NAN;
    return inertia_of(cfg, t_iter);
}

int psops_create(psops_ctx **out, const psops_config *cfg, float *d_x, float *d_v,
                 float *d_pbest, void *d_workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (out == nullptr) return PSOPS_EINVAL;
    *out = nullptr;
    if (!config_ok(cfg) || d_x == nullptr || d_v == nullptr || d_pbest == nullptr) return PSOPS_EINVAL;
    const uintptr_t ax = (uintptr_t)d_x, av = (uintptr_t)d_v, ap = (uintptr_t)d_pbest;
    if ((ax | av | ap) & 3u) return PSOPS_EALIGN;
    const Layout lay = make_layout(cfg);
    if (d_workspace == nullptr || ((uintptr_t)d_workspace & 255u) || workspace_bytes < lay.total)
        return PSOPS_EWORKSPACE;

    psops_ctx *ctx = new (std::nothrow) psops_ctx();
    if (ctx == nullptr) return PSOPS_ENOMEM;
    ctx->cfg = *cfg;
    ctx->lay = lay;
    ctx->x = d_x; ctx->v = d_v; ctx->p = d_pbest;
    ctx->ws = (char *)d_workspace;
    ctx->d_losses = (float *)(ctx->ws + lay.off_losses);
    ctx->loss_src = ctx->d_losses;
    ctx->d_pbest_loss = (float *)(ctx->ws + lay.off_pbest_loss);
    ctx->d_desc = (SyncDesc *)(ctx->ws + lay.off_desc);
    ctx->d_gbest = keeps_gbest(cfg) ? (float *)(ctx->ws + lay.off_gbest) : nullptr;
    ctx->d_snapshot = (keeps_gbest(cfg) || may_split_rows(cfg)) ? (float *)(ctx->ws + lay.off_gbest) : nullptr;
    ctx->row_groups = 1;
    ctx->group_rows = cfg->K;
    ctx->Kt = swarm_size(cfg);
    ctx->selected = false;
    ctx->range_next = 0;
    ctx->h_g = ctx->d_g = nullptr;
    ctx->ev_select = nullptr;
    ctx->d_partials = (cfg->flags & PSOPS_QUADRATIC) ? (double *)(ctx->ws + lay.off_partials) : nullptr;
    ctx->dvec = ctx->tvec = nullptr;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->s_in = ctx->s_out = nullptr;
    ctx->aligned = (((ax | av | ap) & 15u) == 0) && (cfg->ld % 4 == 0);
    ctx->have_losses = false;
    ctx->synced_once = false;
    ctx->step = 0;
    ctx->quads = (cfg->N + 3) / 4;
    ctx->tiles = (cfg->N + kTileElems - 1) / kTileElems;
    ctx->launches = 0;
    ctx->err[0] = '\0';

    int rc = PSOPS_OK;
    cudaError_t e = cudaGetDevice(&ctx->device);
    // Cache policy of the update kernel: as many of the arrays x, v, pbest as fit
    // in the given share of the device's L2 are accessed write-back, so that the
    // next sync finds them there; the rest is streamed (evict-first) past them.
    ctx->resident_arrays = 0;
    if (e == cudaSuccess) {
        int l2_bytes = 0;
        e = cudaDeviceGetAttribute(&l2_bytes, cudaDevAttrL2CacheSize, ctx->device);
        const double array_bytes = 4.0 * (double)cfg->K * (double)cfg->N;
        const double room = (double)l2_bytes * (PSOPS_L2_RESIDENT_PERCENT / 100.0);
        if (e == cudaSuccess) {
            while (ctx->resident_arrays < 3 && (ctx->resident_arrays + 1) * array_bytes <= room)
                ctx->resident_arrays += 1;
#ifdef PSOPS_RESIDENT_FROM_ENV               /* tuning builds only */
            if (const char *forced = std::getenv("PSOPS_RESIDENT")) ctx->resident_arrays = std::atoi(forced);
#endif
        }
    }
    // How many blocks of the single-launch form of a sync run at the same time.
    ctx->one_wave_blocks = 0;
    if (e == cudaSuccess) {
        int sms = 0, per_sm = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->device);
        if (e == cudaSuccess)
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                &per_sm, pick_update_kernel(ctx->aligned, false, true, ctx->resident_arrays, false, cfg->K),
                kUpdateThreads, 0);
        ctx->one_wave_blocks = (long long)sms * per_sm;
        // Rows split into groups when one group per column block would leave most
        // of the GPU idle: as many groups as fit in one wave of the plain kernel,
        // each with at least one full batch of rows.
        if (e == cudaSuccess && may_split_rows(cfg)) {
            int plain_per_sm = 0;
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                &plain_per_sm, pick_update_kernel(ctx->aligned, false, false, ctx->resident_arrays, false, cfg->K, true),
                kUpdateThreads, 0);
            const long long column_blocks = (ctx->quads + (long long)kUpdateThreads * kQuads - 1) / ((long long)kUpdateThreads * kQuads);
            long long groups = (long long)sms * plain_per_sm / column_blocks;
            const long long most = (cfg->K + kSplitRowsPerGroup - 1) / kSplitRowsPerGroup;
            if (groups > most) groups = most;
            if (e == cudaSuccess && groups >= 2) {
                ctx->group_rows = (int)((cfg->K + groups - 1) / groups);
                ctx->row_groups = (cfg->K + ctx->group_rows - 1) / ctx->group_rows;
            }
        }
    }
    if (e == cudaSuccess) {
        // pBest_loss <- +inf (Algorithm 2 clones weights only), descriptor <- 0.
        std::vector<float> inf((size_t)ctx->Kt, INFINITY);
        e = cudaMemcpyAsync(ctx->d_pbest_loss, inf.data(), sizeof(float) * (size_t)ctx->Kt,
                            cudaMemcpyHostToDevice, ctx->stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_desc, 0, sizeof(SyncDesc), ctx->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);   // `inf` is pageable
    }
    if (e != cudaSuccess) {
        rc = PSOPS_ECUDA;
        delete ctx;
        return rc;
    }
    *out = ctx;
    return PSOPS_OK;
}

int psops_set_losses(psops_ctx *ctx, const float *losses, int on_device)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr || losses == nullptr) return PSOPS_EINVAL;
    const size_t bytes = sizeof(float) * (size_t)ctx->Kt;
    if (on_device) {
        if (((uintptr_t)losses & 3u) != 0) return PSOPS_EALIGN;
        ctx->loss_src = losses;        // read (and copied) by the selection kernel of the next sync
    } else {
        const int rc = check_host_losses(losses, ctx->Kt);
        if (rc != PSOPS_OK) return rc;
        // The source may be pageable and may be reused at once: wait for the copy.
        PSOPS_CUDA(ctx, cudaMemcpyAsync(ctx->d_losses, losses, bytes, cudaMemcpyHostToDevice, ctx->stream));
        PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        ctx->loss_src = ctx->d_losses;
    }
    ctx->have_losses = true;
    return PSOPS_OK;
}

int psops_sync(psops_ctx *ctx, int64_t t_iter, float lambda)
{
    DeviceGuard device_guard(ctx);
    int rc = validate_sync_args(ctx, t_iter, lambda);
    if (rc != PSOPS_OK) return rc;
    if (!ctx->have_losses) return PSOPS_ESTATE;
    if (ctx->Kt != ctx->cfg.K) return PSOPS_ESTATE;     // a shard needs gBest from outside: psops_shard_*
    const float m = inertia_of(&ctx->cfg, t_iter);
    const float k1 = ctx->cfg.c1 / lambda;
    const float k2 = ctx->cfg.c2 / lambda;
    const bool fitness = ctx->dvec != nullptr;

    // A small swarm (at most 8 particles, all blocks of the update resident at
    // once) is launch-bound: there the update launch does the selection itself,
    // one kernel per sync.  Anything larger, the history variant and the fused
    // fitness run the selection kernel first and the update behind it, which
    // costs a large grid nothing and keeps its blocks free of the closing step.
    const long long update_blocks = (ctx->quads + (long long)kUpdateThreads * kQuads - 1) / ((long long)kUpdateThreads * kQuads);
    const bool select_in_update = ctx->cfg.K <= kSelectMaxParticles && !fitness &&
                                  update_blocks <= ctx->one_wave_blocks &&
                                  !(ctx->cfg.flags & (PSOPS_GBEST_HISTORY | PSOPS_SEPARATE_SELECT));
    // Many particles on few elements: one thread walking all K rows would leave
    // most SMs idle, so the rows are split into groups over blockIdx.y.  Row g
    // is then read by blocks that do not write it: it is copied to a snapshot
    // first, by a kernel that up to 32 particles also does the selection
    // (snapshot -> update; beyond 32: selection -> snapshot -> update), each
    // launched programmatically behind the other.
    const bool split_rows = ctx->row_groups > 1 && !fitness && !select_in_update;
    const bool select_in_snapshot = split_rows && ctx->cfg.K <= 32 && !(ctx->cfg.flags & PSOPS_SEPARATE_SELECT);
    if (!select_in_update && !select_in_snapshot) {
        rc = launch_select(ctx);
        if (rc != PSOPS_OK) return rc;
    }
    if (select_in_snapshot) {
        const unsigned blocks = (unsigned)((ctx->quads + kUpdateThreads - 1) / kUpdateThreads);
        const cudaError_t e = ctx->aligned
            ? launch_serialized(true, psops_select_snapshot_kernel<true>, dim3(blocks, 1, 1), dim3(kUpdateThreads, 1, 1),
                                ctx->stream, ctx->loss_src, ctx->d_losses, ctx->d_pbest_loss, ctx->d_desc, ctx->cfg.K,
                                (const float *)ctx->x, (long long)ctx->cfg.ld, (long long)ctx->cfg.N, ctx->quads,
                                ctx->d_snapshot)
            : launch_serialized(true, psops_select_snapshot_kernel<false>, dim3(blocks, 1, 1), dim3(kUpdateThreads, 1, 1),
                                ctx->stream, ctx->loss_src, ctx->d_losses, ctx->d_pbest_loss, ctx->d_desc, ctx->cfg.K,
                                (const float *)ctx->x, (long long)ctx->cfg.ld, (long long)ctx->cfg.N, ctx->quads,
                                ctx->d_snapshot);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "psops_select_snapshot_kernel launch");
        ctx->loss_src = ctx->d_losses;              // the kernel keeps a copy there
        rc = check_launch(ctx, "psops_select_snapshot_kernel");
        if (rc != PSOPS_OK) return rc;
    } else if (split_rows) {
        const unsigned blocks = (unsigned)((ctx->quads + kUpdateThreads - 1) / kUpdateThreads);
        const cudaError_t e = ctx->aligned
            ? launch_serialized(true, psops_gbest_snapshot_kernel<true>, dim3(blocks, 1, 1), dim3(kUpdateThreads, 1, 1),
                                ctx->stream, (const SyncDesc *)ctx->d_desc, (const float *)ctx->x,
                                (long long)ctx->cfg.ld, (long long)ctx->cfg.N, ctx->quads, ctx->d_snapshot)
            : launch_serialized(true, psops_gbest_snapshot_kernel<false>, dim3(blocks, 1, 1), dim3(kUpdateThreads, 1, 1),
                                ctx->stream, (const SyncDesc *)ctx->d_desc, (const float *)ctx->x,
                                (long long)ctx->cfg.ld, (long long)ctx->cfg.N, ctx->quads, ctx->d_snapshot);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "psops_gbest_snapshot_kernel launch");
        rc = check_launch(ctx, "psops_gbest_snapshot_kernel");
        if (rc != PSOPS_OK) return rc;
    }
    // With the fused fitness every warp of a tile must be whole: round the
    // quad range up to a tile; quads past the end contribute +0.0.
    const long long q_end = fitness ? ctx->tiles * 32 : ctx->quads;
    rc = launch_update(ctx, m, k1, k2, 0, q_end, fitness, ctx->stream, /*programmatic=*/true, select_in_update,
                       split_rows ? ctx->d_snapshot : nullptr, split_rows);
    if (rc != PSOPS_OK) return rc;
    if (fitness) {
        rc = launch_finalize(ctx);
        if (rc != PSOPS_OK) return rc;
    }
    ctx->step += 1;
    ctx->synced_once = true;
    return PSOPS_OK;
}

// The pipelined body of psops_sync_host; any error leaves copies and kernels
// queued, which the caller below drains before it reports the failure.
static int sync_host_enqueue(psops_ctx *ctx, const float *h_x_in, int64_t h_in_ld, const float *h_losses,
                             float m, float k1, float k2, bool fitness, float *h_x_out, int64_t h_out_ld)
{
    const int K = ctx->cfg.K;
    const long long N = ctx->cfg.N;
    // Losses and selection first: the update of any element range needs them.
    PSOPS_CUDA(ctx, cudaMemcpyAsync(ctx->d_losses, h_losses, sizeof(float) * (size_t)K,
                                    cudaMemcpyHostToDevice, ctx->stream));
    ctx->loss_src = ctx->d_losses;
    ctx->have_losses = true;
    int rc = launch_select(ctx);
    if (rc != PSOPS_OK) return rc;

    // Element ranges of whole tiles, PSOPS_HOST_CHUNK_BYTES of weights per range.
    long long chunk_q = (((long long)PSOPS_HOST_CHUNK_BYTES) / (16ll * K)) / 32 * 32;
    if (chunk_q < 32 * 256) chunk_q = 32 * 256;
    const long long q_total = fitness ? ctx->tiles * 32 : ctx->quads;
    size_t ev = 0;
    cudaEvent_t e_start;
    rc = get_event(ctx, ev++, &e_start);
    if (rc != PSOPS_OK) return rc;
    PSOPS_CUDA(ctx, cudaEventRecord(e_start, ctx->stream));        // earlier work on x is done
    PSOPS_CUDA(ctx, cudaStreamWaitEvent(ctx->s_in, e_start, 0));

    for (long long q0 = 0; q0 < q_total; q0 += chunk_q) {
        const long long q1 = (q0 + chunk_q < q_total) ? q0 + chunk_q : q_total;
        const long long d0 = q0 * 4;
        const long long d1 = (q1 * 4 < N) ? q1 * 4 : N;
        cudaEvent_t e_in, e_k;
        rc = get_event(ctx, ev++, &e_in);
        if (rc != PSOPS_OK) return rc;
        rc = get_event(ctx, ev++, &e_k);
        if (rc != PSOPS_OK) return rc;
        if (d1 > d0) {
            rc = copy_rows(ctx, ctx->x + d0, (size_t)ctx->cfg.ld, h_x_in + d0, (size_t)h_in_ld,
                           (size_t)(d1 - d0), K, cudaMemcpyHostToDevice, ctx->s_in);
            if (rc != PSOPS_OK) return rc;
        }
        PSOPS_CUDA(ctx, cudaEventRecord(e_in, ctx->s_in));
        PSOPS_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, e_in, 0));
        rc = launch_update(ctx, m, k1, k2, q0, q1, fitness, ctx->stream);
        if (rc != PSOPS_OK) return rc;
        PSOPS_CUDA(ctx, cudaEventRecord(e_k, ctx->stream));
        PSOPS_CUDA(ctx, cudaStreamWaitEvent(ctx->s_out, e_k, 0));
        if (d1 > d0) {
            rc = copy_rows(ctx, h_x_out + d0, (size_t)h_out_ld, ctx->x + d0, (size_t)ctx->cfg.ld,
                           (size_t)(d1 - d0), K, cudaMemcpyDeviceToHost, ctx->s_out);
            if (rc != PSOPS_OK) return rc;
        }
    }
    if (fitness) {
        rc = launch_finalize(ctx);
        if (rc != PSOPS_OK) return rc;
    }
    return PSOPS_OK;
}

int psops_sync_host(psops_ctx *ctx, const float *h_x_in, int64_t h_in_ld, const float *h_losses,
                    int64_t t_iter, float lambda, float *h_x_out, int64_t h_out_ld)
{
    DeviceGuard device_guard(ctx);
    int rc = validate_sync_args(ctx, t_iter, lambda);
    if (rc != PSOPS_OK) return rc;
    if (h_x_in == nullptr || h_x_out == nullptr) return PSOPS_EINVAL;
    if (h_in_ld < ctx->cfg.N || h_out_ld < ctx->cfg.N) return PSOPS_EINVAL;
    if (ctx->Kt != ctx->cfg.K) return PSOPS_ESTATE;
    rc = check_host_losses(h_losses, ctx->cfg.K);
    if (rc != PSOPS_OK) return rc;

    const float m = inertia_of(&ctx->cfg, t_iter);
    const float k1 = ctx->cfg.c1 / lambda;
    const float k2 = ctx->cfg.c2 / lambda;
    const bool fitness = ctx->dvec != nullptr;

    if (ctx->s_in == nullptr) {
        PSOPS_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking));
        PSOPS_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking));
    }

    rc = sync_host_enqueue(ctx, h_x_in, h_in_ld, h_losses, m, k1, k2, fitness, h_x_out, h_out_ld);
    // Success or not, nothing may still be in flight against the caller's host
    // buffers when this call returns: wait for both copy streams and the kernels.
    const cudaError_t w_in = cudaStreamSynchronize(ctx->s_in);
    const cudaError_t w_out = cudaStreamSynchronize(ctx->s_out);
    const cudaError_t w_main = cudaStreamSynchronize(ctx->stream);
    if (rc != PSOPS_OK) return rc;          // the state is then undefined: part of the ranges may have been updated
    if (w_in != cudaSuccess) return cuda_fail(ctx, w_in, "psops_sync_host: input copies");
    if (w_out != cudaSuccess) return cuda_fail(ctx, w_out, "psops_sync_host: output copies");
    if (w_main != cudaSuccess) return cuda_fail(ctx, w_main, "psops_sync_host: kernels");
    ctx->step += 1;
    ctx->synced_once = true;
    return PSOPS_OK;
}

int psops_shard_select(psops_ctx *ctx, int *g)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr || g == nullptr) return PSOPS_EINVAL;
    if (!ctx->have_losses) return PSOPS_ESTATE;
    if (ctx->selected) return PSOPS_ESTATE;     // the update of the previous selection is still due (or half done)
    if (ctx->h_g == nullptr) {
        // One word of page-locked host memory that the selection kernel writes
        // directly: the host then needs no copy and no drain of the stream, only
        // the event behind that kernel.
        void *host = nullptr, *dev = nullptr;
        PSOPS_CUDA(ctx, cudaHostAlloc(&host, sizeof(int), cudaHostAllocMapped));
        cudaError_t e = cudaHostGetDevicePointer(&dev, host, 0);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_select, cudaEventDisableTiming);
        if (e != cudaSuccess) {
            cudaFreeHost(host);
            ctx->ev_select = nullptr;
            return cuda_fail(ctx, e, "psops_shard_select: mapped word");
        }
        ctx->h_g = static_cast<int *>(host);
        ctx->d_g = static_cast<int *>(dev);
    }
    const int rc = launch_select(ctx, ctx->d_g);
    if (rc != PSOPS_OK) return rc;
    PSOPS_CUDA(ctx, cudaEventRecord(ctx->ev_select, ctx->stream));
    PSOPS_CUDA(ctx, cudaEventSynchronize(ctx->ev_select));
    *g = *reinterpret_cast<volatile int *>(ctx->h_g);
    ctx->selected = true;
    ctx->range_next = 0;
    ctx->synced_once = true;
    return PSOPS_OK;
}

int psops_shard_update_range(psops_ctx *ctx, int64_t t_iter, float lambda, const float *d_gbest_row,
                             int64_t first_elem, int64_t last_elem)
{
    DeviceGuard device_guard(ctx);
    int rc = validate_sync_args(ctx, t_iter, lambda);
    if (rc != PSOPS_OK) return rc;
    if (d_gbest_row == nullptr) return PSOPS_EINVAL;
    if (((uintptr_t)d_gbest_row & 3u) || (ctx->aligned && ((uintptr_t)d_gbest_row & 15u))) return PSOPS_EALIGN;
    if (!ctx->selected || ctx->dvec != nullptr) return PSOPS_ESTATE;
    const long long N = ctx->cfg.N;
    if (first_elem != ctx->range_next) return PSOPS_ESTATE;             // ranges go left to right without gaps
    if (first_elem < 0 || last_elem <= first_elem || last_elem > N) return PSOPS_EINVAL;
    if ((first_elem & 3) || ((last_elem & 3) && last_elem != N)) return PSOPS_EINVAL;   // whole quads
    const float m = inertia_of(&ctx->cfg, t_iter);
    const float k1 = ctx->cfg.c1 / lambda;
    const float k2 = ctx->cfg.c2 / lambda;
    rc = launch_update(ctx, m, k1, k2, first_elem / 4, (last_elem + 3) / 4, false, ctx->stream,
                       /*programmatic=*/false, /*select=*/false, d_gbest_row);
    if (rc != PSOPS_OK) return rc;
    ctx->range_next = last_elem;
    if (last_elem == N) {                   // the sync is complete
        ctx->selected = false;
        ctx->range_next = 0;
        ctx->step += 1;
    }
    return PSOPS_OK;
}

int psops_shard_update(psops_ctx *ctx, int64_t t_iter, float lambda, const float *d_gbest_row)
{
    if (ctx == nullptr) return PSOPS_EINVAL;
    return psops_shard_update_range(ctx, t_iter, lambda, d_gbest_row, 0, ctx->cfg.N);
}

int psops_ssgd(psops_ctx *ctx, const float *d_grad, int64_t grad_ld, float alpha)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr || d_grad == nullptr || grad_ld < ctx->cfg.N || !std::isfinite(alpha)) return PSOPS_EINVAL;
    if (ctx->Kt != ctx->cfg.K) return PSOPS_ESTATE;     // the mean runs over the whole swarm, a shard holds a part
    if ((uintptr_t)d_grad & 3u) return PSOPS_EALIGN;
    const float scale = alpha / (float)ctx->cfg.K;
    const unsigned blocks = (unsigned)((ctx->quads + kUpdateThreads - 1) / kUpdateThreads);
    const bool aligned = ctx->aligned && (((uintptr_t)d_grad & 15u) == 0) && (grad_ld % 4 == 0);
    if (aligned)
        psops_ssgd_kernel<true, 8><<<blocks, kUpdateThreads, 0, ctx->stream>>>(
            ctx->x, d_grad, ctx->cfg.ld, grad_ld, ctx->cfg.N, ctx->quads, ctx->cfg.K, scale);
    else
        psops_ssgd_kernel<false, 8><<<blocks, kUpdateThreads, 0, ctx->stream>>>(
            ctx->x, d_grad, ctx->cfg.ld, grad_ld, ctx->cfg.N, ctx->quads, ctx->cfg.K, scale);
    return check_launch(ctx, "psops_ssgd_kernel");
}

int psops_get_history(psops_ctx *ctx, float *gbest_loss, int *valid)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr) return PSOPS_EINVAL;
    if (!(ctx->cfg.flags & PSOPS_GBEST_HISTORY)) return PSOPS_ESTATE;
    SyncDesc host{};
    PSOPS_CUDA(ctx, cudaMemcpyAsync(&host, ctx->d_desc, sizeof(SyncDesc), cudaMemcpyDeviceToHost, ctx->stream));
    PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (gbest_loss != nullptr) *gbest_loss = host.hist_loss;
    if (valid != nullptr) *valid = host.hist_valid;
    return PSOPS_OK;
}

int psops_set_history(psops_ctx *ctx, float gbest_loss, const float *gbest_row, int row_on_device)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr || gbest_row == nullptr) return PSOPS_EINVAL;
    if (!(ctx->cfg.flags & PSOPS_GBEST_HISTORY)) return PSOPS_ESTATE;
    if (gbest_loss != gbest_loss) return PSOPS_ENAN;
    const int one = 1;
    char *desc = reinterpret_cast<char *>(ctx->d_desc);
    PSOPS_CUDA(ctx, cudaMemcpyAsync(ctx->d_gbest, gbest_row, sizeof(float) * (size_t)ctx->cfg.N,
                                    row_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, ctx->stream));
    PSOPS_CUDA(ctx, cudaMemcpyAsync(desc + offsetof(SyncDesc, hist_loss), &gbest_loss, sizeof(float),
                                    cudaMemcpyHostToDevice, ctx->stream));
    PSOPS_CUDA(ctx, cudaMemcpyAsync(desc + offsetof(SyncDesc, hist_valid), &one, sizeof(int),
                                    cudaMemcpyHostToDevice, ctx->stream));
    PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    ctx->synced_once = true;           // PSOPS_GBEST can be read back
    return PSOPS_OK;
}

int psops_host_register(void *host_ptr, size_t bytes)
{
    if (host_ptr == nullptr || bytes == 0) return PSOPS_EINVAL;
    const cudaError_t e = cudaHostRegister(host_ptr, bytes, cudaHostRegisterDefault);
    if (e == cudaErrorHostMemoryAlreadyRegistered) {
        (void)cudaGetLastError();
        return PSOPS_OK;
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return PSOPS_ECUDA;
    }
    return PSOPS_OK;
}

int psops_host_unregister(void *host_ptr)
{
    if (host_ptr == nullptr) return PSOPS_EINVAL;
    if (cudaHostUnregister(host_ptr) != cudaSuccess) {
        (void)cudaGetLastError();
        return PSOPS_ECUDA;
    }
    return PSOPS_OK;
}

int psops_average(psops_ctx *ctx)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr) return PSOPS_EINVAL;
    if (ctx->Kt != ctx->cfg.K) return PSOPS_ESTATE;     // the mean runs over the whole swarm, a shard holds a part
    const unsigned blocks = (unsigned)((ctx->quads + kUpdateThreads - 1) / kUpdateThreads);
    if (ctx->aligned)
        psops_average_kernel<true, 8><<<blocks, kUpdateThreads, 0, ctx->stream>>>(
            ctx->x, ctx->cfg.ld, ctx->cfg.N, ctx->quads, ctx->cfg.K);
    else
        psops_average_kernel<false, 8><<<blocks, kUpdateThreads, 0, ctx->stream>>>(
            ctx->x, ctx->cfg.ld, ctx->cfg.N, ctx->quads, ctx->cfg.K);
    return check_launch(ctx, "psops_average_kernel");
}

static int row_pointer(psops_ctx *ctx, int which, int k, float **row)
{
    if (which == PSOPS_GBEST) {
        if (ctx->d_gbest == nullptr || !ctx->synced_once) return PSOPS_ESTATE;
        *row = ctx->d_gbest;
        return PSOPS_OK;
    }
    if (k < 0 || k >= ctx->cfg.K) return PSOPS_EINVAL;
    float *base = which == PSOPS_X ? ctx->x : which == PSOPS_V ? ctx->v : which == PSOPS_PBEST ? ctx->p : nullptr;
    if (base == nullptr) return PSOPS_EINVAL;
    *row = base + (size_t)k * (size_t)ctx->cfg.ld;
    return PSOPS_OK;
}

int psops_get_weights(psops_ctx *ctx, int which, int k, float *dst, int dst_on_device)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr || dst == nullptr) return PSOPS_EINVAL;
    float *row = nullptr;
    const int rc = row_pointer(ctx, which, k, &row);
    if (rc != PSOPS_OK) return rc;
    const size_t bytes = sizeof(float) * (size_t)ctx->cfg.N;
    PSOPS_CUDA(ctx, cudaMemcpyAsync(dst, row, bytes,
                                    dst_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost,
                                    ctx->stream));
    if (!dst_on_device) PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return PSOPS_OK;
}

int psops_set_weights(psops_ctx *ctx, int which, int k, const float *src, int src_on_device)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr || src == nullptr) return PSOPS_EINVAL;
    if (which == PSOPS_GBEST) return PSOPS_EINVAL;
    float *row = nullptr;
    const int rc = row_pointer(ctx, which, k, &row);
    if (rc != PSOPS_OK) return rc;
    const size_t bytes = sizeof(float) * (size_t)ctx->cfg.N;
    PSOPS_CUDA(ctx, cudaMemcpyAsync(row, src, bytes,
                                    src_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice,
                                    ctx->stream));
    if (!src_on_device) PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return PSOPS_OK;
}

int psops_sync_info(psops_ctx *ctx, int *g, uint32_t *improved_words, float *pbest_loss)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr) return PSOPS_EINVAL;
    if (!ctx->synced_once) return PSOPS_ESTATE;
    SyncDesc host{};
    PSOPS_CUDA(ctx, cudaMemcpyAsync(&host, ctx->d_desc, sizeof(SyncDesc), cudaMemcpyDeviceToHost, ctx->stream));
    if (pbest_loss != nullptr)
        PSOPS_CUDA(ctx, cudaMemcpyAsync(pbest_loss, ctx->d_pbest_loss, sizeof(float) * (size_t)ctx->Kt,
                                        cudaMemcpyDeviceToHost, ctx->stream));
    PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (g != nullptr) *g = host.g;
    if (improved_words != nullptr)
        std::memcpy(improved_words, host.improved, sizeof(uint32_t) * (size_t)((ctx->Kt + 31) / 32));
    return PSOPS_OK;
}

int psops_get_losses(psops_ctx *ctx, float *dst, int dst_on_device)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr || dst == nullptr) return PSOPS_EINVAL;
    if (!ctx->have_losses) return PSOPS_ESTATE;
    PSOPS_CUDA(ctx, cudaMemcpyAsync(dst, ctx->loss_src, sizeof(float) * (size_t)ctx->Kt,
                                    dst_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost,
                                    ctx->stream));
    if (!dst_on_device) PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return PSOPS_OK;
}

int psops_set_quadratic(psops_ctx *ctx, const float *d_dvec, const float *d_tvec)
{
    if (ctx == nullptr) return PSOPS_EINVAL;
    if (d_dvec == nullptr && d_tvec == nullptr) {
        ctx->dvec = ctx->tvec = nullptr;
        return PSOPS_OK;
    }
    if (d_dvec == nullptr || d_tvec == nullptr) return PSOPS_EINVAL;
    if (ctx->d_partials == nullptr) return PSOPS_EWORKSPACE;
    if (((uintptr_t)d_dvec | (uintptr_t)d_tvec) & 3u) return PSOPS_EALIGN;
    // the 128-bit path also reads dvec/tvec as quads
    if (ctx->aligned && (((uintptr_t)d_dvec | (uintptr_t)d_tvec) & 15u)) return PSOPS_EALIGN;
    ctx->dvec = d_dvec;
    ctx->tvec = d_tvec;
    return PSOPS_OK;
}

int psops_eval_quadratic(psops_ctx *ctx)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr) return PSOPS_EINVAL;
    if (ctx->dvec == nullptr) return PSOPS_ESTATE;
    const long long threads = ctx->tiles * 32;
    const unsigned blocks = (unsigned)((threads + kUpdateThreads - 1) / kUpdateThreads);
    if (ctx->aligned)
        psops_fitness_tiles_kernel<true><<<blocks, kUpdateThreads, 0, ctx->stream>>>(
            ctx->x, ctx->dvec, ctx->tvec, ctx->d_partials, ctx->cfg.ld, ctx->cfg.N, ctx->quads,
            ctx->tiles, ctx->cfg.K);
    else
        psops_fitness_tiles_kernel<false><<<blocks, kUpdateThreads, 0, ctx->stream>>>(
            ctx->x, ctx->dvec, ctx->tvec, ctx->d_partials, ctx->cfg.ld, ctx->cfg.N, ctx->quads,
            ctx->tiles, ctx->cfg.K);
    int rc = check_launch(ctx, "psops_fitness_tiles_kernel");
    if (rc != PSOPS_OK) return rc;
    rc = launch_finalize(ctx);
    if (rc != PSOPS_OK) return rc;
    ctx->have_losses = true;
    return PSOPS_OK;
}

int psops_get_state(psops_ctx *ctx, uint32_t *sync_step, float *pbest_loss)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr) return PSOPS_EINVAL;
    // The counter lives on the device (a replayed graph advances it without
    // the host taking part), so read it from there.
    SyncDesc host{};
    PSOPS_CUDA(ctx, cudaMemcpyAsync(&host, ctx->d_desc, sizeof(SyncDesc), cudaMemcpyDeviceToHost, ctx->stream));
    if (pbest_loss != nullptr)
        PSOPS_CUDA(ctx, cudaMemcpyAsync(pbest_loss, ctx->d_pbest_loss, sizeof(float) * (size_t)ctx->Kt,
                                        cudaMemcpyDeviceToHost, ctx->stream));
    PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    ctx->step = host.next_step;
    if (sync_step != nullptr) *sync_step = host.next_step;
    return PSOPS_OK;
}

int psops_set_state(psops_ctx *ctx, uint32_t sync_step, const float *pbest_loss)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr || pbest_loss == nullptr) return PSOPS_EINVAL;
    for (int i = 0; i < ctx->Kt; ++i)
        if (pbest_loss[i] != pbest_loss[i]) return PSOPS_ENAN;
    PSOPS_CUDA(ctx, cudaMemcpyAsync(ctx->d_pbest_loss, pbest_loss, sizeof(float) * (size_t)ctx->Kt,
                                    cudaMemcpyHostToDevice, ctx->stream));
    PSOPS_CUDA(ctx, cudaMemcpyAsync(reinterpret_cast<char *>(ctx->d_desc) + offsetof(SyncDesc, next_step),
                                    &sync_step, sizeof(uint32_t), cudaMemcpyHostToDevice, ctx->stream));
    PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    ctx->step = sync_step;
    return PSOPS_OK;
}

int64_t psops_launch_count(const psops_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *psops_strerror(int code)
{
    switch (code) {
    case PSOPS_OK: return "ok";
    case PSOPS_EINVAL: return "invalid argument";
    case PSOPS_EALIGN: return "device pointer not sufficiently aligned";
    case PSOPS_ESTATE: return "call not valid in the current state";
    case PSOPS_ENAN: return "NaN in host-supplied losses";
    case PSOPS_EWORKSPACE: return "workspace missing, misaligned or too small";
    case PSOPS_ECUDA: return "CUDA call failed";
    case PSOPS_ENOMEM: return "host allocation failed";
    case PSOPS_ELIMIT: return "problem larger than the library's built-in scratch array";
    default: return "unknown error code";
    }
}

const char *psops_last_error(const psops_ctx *ctx) { return ctx ? ctx->err : ""; }

int psops_destroy(psops_ctx *ctx)
{
    DeviceGuard device_guard(ctx);
    if (ctx == nullptr) return PSOPS_EINVAL;
    int rc = PSOPS_OK;
    if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) rc = PSOPS_ECUDA;
    for (cudaEvent_t e : ctx->events) cudaEventDestroy(e);
    if (ctx->s_in) cudaStreamDestroy(ctx->s_in);
    if (ctx->s_out) cudaStreamDestroy(ctx->s_out);
    if (ctx->ev_select) cudaEventDestroy(ctx->ev_select);
    if (ctx->h_g) cudaFreeHost(ctx->h_g);
    delete ctx;
    return rc;
}

} // extern "C"

// ---------------------------------------------------------------------------
// Allocation-free fitness evaluation.
//
// Some callers cannot obtain device memory at the moment they need a fitness
// value: code running inside a serving or training loop whose framework has
// already handed every byte of the GPU to its own caching allocator, plug-ins
// that are only given input and output buffers, and latency-critical loops
// that must not call cudaMalloc / cudaFree because those calls synchronise the
// whole device.  For them the tile sums of the quadratic fitness live in a
// fixed array that is part of this library's device image instead of in a
// caller-provided workspace.
//
// The array costs PSOPS_STATIC_SCRATCH_DOUBLES * 8 bytes (8 MiB) on every GPU
// that loads the library, for the life of the process.  All calls on a device
// share it and it keeps whatever the previous call left there; the finaliser
// reads only slots that the tile kernel of the same call has just written, so
// nothing needs clearing.  Two calls that run concurrently on one GPU (two
// streams, two host threads) would overwrite each other's tile sums.
// ---------------------------------------------------------------------------
static __device__ __align__(256) double psops_static_tile_sums[PSOPS_STATIC_SCRATCH_DOUBLES];

namespace {

constexpr int kMaxDevices = 64;
double *g_static_tile_sums[kMaxDevices];      // device address of the array, per device ordinal
bool g_static_ready[kMaxDevices];
std::mutex g_static_mutex;

// `psops_static_tile_sums` in host code is only a handle for the runtime, not
// an address a kernel can use: resolve it once per device, with that device
// current, and hand the result to the kernels.
int static_scratch_for_current_device(double **ptr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSOPS_ECUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ready[dev]) {
        void *addr = nullptr;
        if (cudaGetSymbolAddress(&addr, psops_static_tile_sums) != cudaSuccess || addr == nullptr) {
            (void)cudaGetLastError();
            return PSOPS_ECUDA;
        }
        g_static_tile_sums[dev] = static_cast<double *>(addr);
        g_static_ready[dev] = true;
    }
    *ptr = g_static_tile_sums[dev];
    return PSOPS_OK;
}

} // namespace

extern "C" int psops_quadratic_fitness_static(const float *d_x, int64_t ld, int32_t K, int64_t N,
                                              const float *d_dvec, const float *d_tvec,
                                              float *d_loss, void *cuda_stream)
{
    if (d_x == nullptr || d_dvec == nullptr || d_tvec == nullptr || d_loss == nullptr) return PSOPS_EINVAL;
    if (K < 1 || K > PSOPS_MAX_K || N < 1 || N >= (1ll << 33) || ld < N) return PSOPS_EINVAL;
    const uintptr_t bits = (uintptr_t)d_x | (uintptr_t)d_dvec | (uintptr_t)d_tvec;
    if ((bits & 3u) || ((uintptr_t)d_loss & 3u)) return PSOPS_EALIGN;
    const long long tiles = (N + kTileElems - 1) / kTileElems;
    if ((long long)K * tiles > (long long)PSOPS_STATIC_SCRATCH_DOUBLES) return PSOPS_ELIMIT;

    // The built-in array that is used is the current device's: the buffers must
    // live there too (a pointer the runtime does not know, e.g. one from another
    // allocator it cannot see, is let through).
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess) return PSOPS_ECUDA;
    const void *buffers[4] = {d_x, d_dvec, d_tvec, d_loss};
    for (const void *ptr : buffers) {
        cudaPointerAttributes where{};
        if (cudaPointerGetAttributes(&where, ptr) != cudaSuccess) {
            (void)cudaGetLastError();
            continue;
        }
        if (where.type == cudaMemoryTypeHost) return PSOPS_EINVAL;
        if (where.type == cudaMemoryTypeDevice && where.device != current) return PSOPS_EINVAL;
    }

    double *tile_sums = nullptr;
    const int rc = static_scratch_for_current_device(&tile_sums);
    if (rc != PSOPS_OK) return rc;

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const long long quads = (N + 3) / 4;
    const unsigned blocks = (unsigned)((tiles * 32 + kUpdateThreads - 1) / kUpdateThreads);
    const bool aligned = ((bits & 15u) == 0) && (ld % 4 == 0);
    if (aligned)
        psops_fitness_tiles_kernel<true><<<blocks, kUpdateThreads, 0, stream>>>(
            d_x, d_dvec, d_tvec, tile_sums, ld, N, quads, tiles, K);
    else
        psops_fitness_tiles_kernel<false><<<blocks, kUpdateThreads, 0, stream>>>(
            d_x, d_dvec, d_tvec, tile_sums, ld, N, quads, tiles, K);
    if (cudaGetLastError() != cudaSuccess) return PSOPS_ECUDA;
    psops_fitness_finalize_kernel<<<dim3(kFinalizeCluster, K), kFinalizeCtaThreads, 0, stream>>>(tile_sums, d_loss, tiles);
    if (cudaGetLastError() != cudaSuccess) return PSOPS_ECUDA;
    return PSOPS_OK;
}
