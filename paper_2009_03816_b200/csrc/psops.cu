// psops.cu -- sm_100a kernels and C ABI of the PSO-PS synchronisation stage.
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

#include <cuda_runtime.h>

#include <cmath>
#include <cstddef>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

namespace {

// ---------------------------------------------------------------------------
// Device-side data
// ---------------------------------------------------------------------------

// Result of the selection kernel, read by the update kernel.
struct SyncDesc {
    int      g;                 // index of the gBest particle (Algorithm 3)
    uint32_t step;              // sync counter s of the sync in progress (Philox counter word 2)
    uint32_t next_step;         // s of the next sync; advanced by the selection kernel so that a
                                // captured-and-replayed sync still walks the random stream
    int      pad;
    uint32_t improved[PSOPS_MAX_K / 32];   // bit i: loss_i < pBest_loss_i
};

struct UpdateParams {
    float *x, *v, *p;           // K rows of stride ld
    float *gbest_copy;          // NULL or N floats
    const float *dvec, *tvec;   // quadratic fitness vectors (FITNESS only)
    double *partials;           // K x tiles tile sums (FITNESS only)
    const SyncDesc *desc;
    long long ld, N;
    long long q_begin, q_end;   // quad range of this launch (quad = 4 elements)
    long long tiles;            // ceil(N / 128)
    int K;
    float m, k1, k2;            // inertia, c1/lambda, c2/lambda
    uint32_t rk[20];            // Philox round keys, rk[2r], rk[2r+1]
};

// Launch shape of the streaming kernels; the defaults are the measured best on
// B200 and can be overridden at build time for tuning sweeps.
#ifndef PSOPS_UPDATE_THREADS
#define PSOPS_UPDATE_THREADS 256
#endif
#ifndef PSOPS_UPDATE_UNROLL
#define PSOPS_UPDATE_UNROLL 4          // particles in flight per thread; must divide 32
#endif
#ifndef PSOPS_UPDATE_QUADS
#define PSOPS_UPDATE_QUADS 1           // quads per thread, one block-width apart
#endif
#ifndef PSOPS_FITNESS_UNROLL
#define PSOPS_FITNESS_UNROLL 2         // particles in flight when the fitness is fused in
#endif
#ifndef PSOPS_FITNESS_QUADS
#define PSOPS_FITNESS_QUADS 1
#endif
#ifndef PSOPS_UPDATE_MIN_BLOCKS
#define PSOPS_UPDATE_MIN_BLOCKS 0      // >0: resident blocks per SM the register allocation must allow
#endif
#if PSOPS_UPDATE_MIN_BLOCKS > 0
#define PSOPS_UPDATE_BOUNDS __launch_bounds__(PSOPS_UPDATE_THREADS, PSOPS_UPDATE_MIN_BLOCKS)
#else
#define PSOPS_UPDATE_BOUNDS __launch_bounds__(PSOPS_UPDATE_THREADS)
#endif
constexpr int kUpdateThreads = PSOPS_UPDATE_THREADS;
constexpr int kFinalizeThreads = 1024;     // = number of level-2 slots
constexpr int kTileElems = 128;            // one warp x one quad per lane

// Philox4x32-10 (Salmon et al., SC'11).  Round keys are precomputed on the
// host: they are the same for every thread of a launch.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2,
                                              uint32_t c3, const uint32_t (&rk)[20],
                                              uint32_t (&out)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const unsigned long long pa = (unsigned long long)0xD2511F53u * c0;
        const unsigned long long pb = (unsigned long long)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(pb >> 32) ^ c1 ^ rk[2 * r];
        const uint32_t n2 = (uint32_t)(pa >> 32) ^ c3 ^ rk[2 * r + 1];
        c1 = (uint32_t)pb;
        c3 = (uint32_t)pa;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// 32 random bits -> uniform on the 2^24 grid of [0,1); both steps are exact.
__device__ __forceinline__ float uniform24(uint32_t w)
{
    return __fmul_rn(__uint2float_rn(w >> 8), 0x1p-24f);
}

// Load / store of one quad.  nvalid = 4 on the vector path means a full
// 128-bit access; anything else goes element by element under a bound.
template <bool ALIGNED>
__device__ __forceinline__ void load_quad(const float *ptr, int nvalid, float (&a)[4])
{
    if (ALIGNED && nvalid == 4) {
        const float4 t = __ldcs(reinterpret_cast<const float4 *>(ptr));
        a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) a[e] = (e < nvalid) ? __ldcs(ptr + e) : 0.0f;
    }
}

// Plain (cacheable) variant for data that several reads share (gBest row,
// dvec, tvec).
template <bool ALIGNED>
__device__ __forceinline__ void load_quad_cached(const float *ptr, int nvalid, float (&a)[4])
{
    if (ALIGNED && nvalid == 4) {
        const float4 t = *reinterpret_cast<const float4 *>(ptr);
        a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) a[e] = (e < nvalid) ? ptr[e] : 0.0f;
    }
}

template <bool ALIGNED>
__device__ __forceinline__ void store_quad(float *ptr, int nvalid, const float (&a)[4])
{
    if (ALIGNED && nvalid == 4) {
        __stcs(reinterpret_cast<float4 *>(ptr), make_float4(a[0], a[1], a[2], a[3]));
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (e < nvalid) __stcs(ptr + e, a[e]);
    }
}

// Level 0 and level 1 of the canonical fitness sum for one quad per lane:
// fp32 terms dvec*(e*e), widened, added left to right, then the xor butterfly
// over the warp.  Every lane returns the tile sum.
__device__ __forceinline__ double fitness_tile_sum(const float (&xn)[4], const float (&dv)[4],
                                                   const float (&tv)[4], int nvalid)
{
    double q = 0.0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        double term = 0.0;
        if (e < nvalid) {
            const float err = __fsub_rn(xn[e], tv[e]);
            term = (double)__fmul_rn(dv[e], __fmul_rn(err, err));
        }
        q = (e == 0) ? term : __dadd_rn(q, term);
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1)
        q = __dadd_rn(q, __shfl_xor_sync(0xffffffffu, q, off));
    return q;
}

// ---------------------------------------------------------------------------
// Kernel (a): selection.  One block, blockDim = K rounded up to a warp.
// g = argmin loss (lowest index among equal minima, NaN never beats a number);
// improved_i = loss_i < pBest_loss_i; pBest_loss_i <- loss_i where improved.
// (Algorithm 3; Algorithm 1, pBest branch.)
// ---------------------------------------------------------------------------
struct Candidate { float loss; int idx; };

__device__ __forceinline__ bool beats(const Candidate &a, const Candidate &b)
{
    const bool an = a.loss != a.loss, bn = b.loss != b.loss;
    if (an != bn) return bn;                 // a number beats a NaN
    if (!an) {
        if (a.loss < b.loss) return true;
        if (b.loss < a.loss) return false;
    }
    return a.idx < b.idx;                    // equal (or both NaN): lowest index
}

__global__ void __launch_bounds__(PSOPS_MAX_K)
psops_select_kernel(const float *loss, float *loss_keep, float *__restrict__ pbest_loss,
                    SyncDesc *__restrict__ desc, int K)
{
    // Let the update kernel that follows in the stream start its prologue; it
    // waits for this grid to finish before it reads the descriptor.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    __shared__ Candidate warp_best[PSOPS_MAX_K / 32];
    const int i = threadIdx.x;
    const int lane = i & 31, warp = i >> 5;
    const bool live = i < K;
    const float li = live ? loss[i] : 0.0f;
    if (live) loss_keep[i] = li;             // the context's own copy (loss may be the caller's buffer)

    // pBest branch: strict "<" so that an equal loss never replaces pBest.
    const bool improved = live && (li < pbest_loss[i]);
    if (improved) pbest_loss[i] = li;
    const uint32_t word = __ballot_sync(0xffffffffu, improved);
    if (lane == 0) desc->improved[warp] = word;

    // argmin
    Candidate c;
    c.loss = li;
    c.idx = live ? i : 0x7fffffff;
    if (!live) c.loss = __int_as_float(0x7fc00000);      // NaN with the largest index: never wins
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        Candidate o;
        o.loss = __shfl_xor_sync(0xffffffffu, c.loss, off);
        o.idx = __shfl_xor_sync(0xffffffffu, c.idx, off);
        if (beats(o, c)) c = o;
    }
    if (lane == 0) warp_best[warp] = c;
    __syncthreads();
    if (i == 0) {
        const int warps = (blockDim.x + 31) >> 5;
        for (int w = 1; w < warps; ++w)
            if (beats(warp_best[w], c)) c = warp_best[w];
        desc->g = c.idx;
        const uint32_t s_now = desc->next_step;
        desc->step = s_now;
        desc->next_step = s_now + 1u;
    }
}

// ---------------------------------------------------------------------------
// Kernel (b): fused update (Eq. 6, Eq. 7 and the pBest copy of Algorithm 1),
// optionally with the fitness of the new weights (levels 0 and 1).
// A thread owns Q quads (quad q = elements 4q..4q+3), one block-width apart,
// for all K particles; a warp covers one 128-element tile per quad slot.
// U particles x Q quads are in flight per thread: U*Q*3 independent 128-bit
// loads before the first use.  Q > 1 makes every block stream a longer
// contiguous piece of each row, which is what DRAM and the TLB like when K
// rows x 3 arrays are all being walked at once.
// ---------------------------------------------------------------------------
template <bool ALIGNED, bool FITNESS, int U, int Q>
__global__ void PSOPS_UPDATE_BOUNDS
psops_update_kernel(const __grid_constant__ UpdateParams P)
{
    const long long q0 = P.q_begin + (long long)blockIdx.x * (kUpdateThreads * Q) + threadIdx.x;
    // Launched with programmatic stream serialisation right behind the selection
    // kernel: everything that kernel wrote is visible after this wait (a no-op
    // for an ordinary launch).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!FITNESS && q0 >= P.q_end) return;   // with FITNESS whole warps stay for the shuffles

    bool active[Q];
    int nvalid[Q];
    size_t col[Q];                           // element offset of quad slot j inside a row
#pragma unroll
    for (int j = 0; j < Q; ++j) {
        const long long q = q0 + (long long)j * kUpdateThreads;
        const long long d0 = q * 4;
        active[j] = q < P.q_end;
        nvalid[j] = 0;
        if (active[j] && d0 < P.N) nvalid[j] = (P.N - d0 >= 4) ? 4 : (int)(P.N - d0);
        col[j] = (size_t)d0;
    }

    // gBest = row g as it is BEFORE this sync overwrites it; this thread is the
    // only writer of these elements, so reading them first is enough.
    const int g = P.desc->g;
    const uint32_t step = P.desc->step;
    float gb[Q][4];
    float dv[Q][4], tv[Q][4];
#pragma unroll
    for (int j = 0; j < Q; ++j) {
        load_quad_cached<ALIGNED>(P.x + (size_t)g * (size_t)P.ld + col[j], nvalid[j], gb[j]);
        if (P.gbest_copy != nullptr) store_quad<ALIGNED>(P.gbest_copy + col[j], nvalid[j], gb[j]);
        if (FITNESS) {
            load_quad_cached<ALIGNED>(P.dvec + col[j], nvalid[j], dv[j]);
            load_quad_cached<ALIGNED>(P.tvec + col[j], nvalid[j], tv[j]);
        }
    }

    // Philox counter word 0 = element >> 1: 2q for elements 4q, 4q+1 and
    // 2q + 1 for elements 4q+2, 4q+3.
    const uint32_t pair0 = (uint32_t)(2 * q0);

    size_t row = 0;                          // offset of row i0
    uint32_t impw = 0;
    for (int i0 = 0; i0 < P.K; i0 += U) {
        if ((i0 & 31) == 0) impw = P.desc->improved[i0 >> 5];

        float xo[U][Q][4], vo[U][Q][4], pp[U][Q][4];
        bool imp[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + u;
            imp[u] = (impw >> (i & 31)) & 1u;
            if (i < P.K) {
#pragma unroll
                for (int j = 0; j < Q; ++j) {
                    const size_t at = row + (size_t)u * (size_t)P.ld + col[j];
                    load_quad<ALIGNED>(P.x + at, nvalid[j], xo[u][j]);
                    load_quad<ALIGNED>(P.v + at, nvalid[j], vo[u][j]);
                    if (!imp[u]) load_quad<ALIGNED>(P.p + at, nvalid[j], pp[u][j]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + u;
            if (i < P.K) {
#pragma unroll
                for (int j = 0; j < Q; ++j) {
                    const size_t at = row + (size_t)u * (size_t)P.ld + col[j];
                    const uint32_t pair = pair0 + (uint32_t)(2 * j * kUpdateThreads);
                    uint32_t ra[4], rb[4];
                    philox4x32_10(pair, (uint32_t)i, step, 0u, P.rk, ra);
                    philox4x32_10(pair + 1u, (uint32_t)i, step, 0u, P.rk, rb);
                    const uint32_t w1[4] = {ra[0], ra[2], rb[0], rb[2]};   // r1 of elements 0..3
                    const uint32_t w2[4] = {ra[1], ra[3], rb[1], rb[3]};   // r2 of elements 0..3
                    float vn[4], xn[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float w = xo[u][j][e];
                        const float pbest = imp[u] ? w : pp[u][j][e];      // pBest_i = w_i if improved
                        const float dl = __fsub_rn(pbest, w);
                        const float dg = __fsub_rn(gb[j][e], w);
                        const float t1 = __fmul_rn(P.k1, uniform24(w1[e]));
                        const float t2 = __fmul_rn(P.k2, uniform24(w2[e]));
                        const float a0 = __fmul_rn(P.m, vo[u][j][e]);
                        vn[e] = __fmaf_rn(t2, dg, __fmaf_rn(t1, dl, a0));  // Eq. 6
                        xn[e] = __fadd_rn(w, vn[e]);                        // Eq. 7
                    }
                    store_quad<ALIGNED>(P.v + at, nvalid[j], vn);
                    store_quad<ALIGNED>(P.x + at, nvalid[j], xn);
                    if (imp[u]) store_quad<ALIGNED>(P.p + at, nvalid[j], xo[u][j]);
                    if (FITNESS) {
                        const double wsum = fitness_tile_sum(xn, dv[j], tv[j], nvalid[j]);
                        if ((threadIdx.x & 31) == 0 && active[j])   // q_end is a whole number of tiles
                            P.partials[(size_t)i * (size_t)P.tiles + (col[j] >> 7)] = wsum;
                    }
                }
            }
        }
        row += (size_t)U * (size_t)P.ld;
    }
}

// ---------------------------------------------------------------------------
// Kernel (c): parameter averaging (Section II-B, step 5).
// ---------------------------------------------------------------------------
template <bool ALIGNED, int U>
__global__ void __launch_bounds__(kUpdateThreads)
psops_average_kernel(float *__restrict__ x, long long ld, long long N, long long quads, int K)
{
    const long long q = (long long)blockIdx.x * kUpdateThreads + threadIdx.x;
    if (q >= quads) return;
    const long long d0 = q * 4;
    const int nvalid = (N - d0 >= 4) ? 4 : (int)(N - d0);
    const float kf = (float)K;

    float acc[4];
    load_quad<ALIGNED>(x + d0, nvalid, acc);
    int k = 1;
    for (; k < K; k += U) {
        float t[U][4];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (k + u < K) load_quad<ALIGNED>(x + (size_t)(k + u) * (size_t)ld + d0, nvalid, t[u]);
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (k + u < K) {
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[e] = __fadd_rn(acc[e], t[u][e]);
            }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = __fdiv_rn(acc[e], kf);
    for (k = 0; k < K; ++k) store_quad<ALIGNED>(x + (size_t)k * (size_t)ld + d0, nvalid, acc);
}

// ---------------------------------------------------------------------------
// Kernel (d): stand-alone fitness tile sums (levels 0 and 1), and the level-2
// finalisation shared with the fused path.
// ---------------------------------------------------------------------------
template <bool ALIGNED>
__global__ void __launch_bounds__(kUpdateThreads)
psops_fitness_tiles_kernel(const float *__restrict__ x, const float *__restrict__ dvec,
                           const float *__restrict__ tvec, double *__restrict__ partials,
                           long long ld, long long N, long long quads, long long tiles, int K)
{
    const long long q = (long long)blockIdx.x * kUpdateThreads + threadIdx.x;
    const long long d0 = q * 4;
    int nvalid = 0;
    if (q < quads) nvalid = (N - d0 >= 4) ? 4 : (int)(N - d0);
    if ((q >> 5) >= tiles) return;           // whole warp out of range
    float dv[4], tv[4];
    load_quad_cached<ALIGNED>(dvec + d0, nvalid, dv);
    load_quad_cached<ALIGNED>(tvec + d0, nvalid, tv);
    for (int i = 0; i < K; ++i) {
        float xi[4];
        load_quad<ALIGNED>(x + (size_t)i * (size_t)ld + d0, nvalid, xi);
        const double w = fitness_tile_sum(xi, dv, tv, nvalid);
        if ((threadIdx.x & 31) == 0) partials[(size_t)i * (size_t)tiles + (size_t)(q >> 5)] = w;
    }
}

// One block per particle, thread tau = slot tau.
__global__ void __launch_bounds__(kFinalizeThreads)
psops_fitness_finalize_kernel(const double *__restrict__ partials, float *__restrict__ loss,
                              long long tiles)
{
    __shared__ double group[kFinalizeThreads / 32];
    const int i = blockIdx.x;
    const double *row = partials + (size_t)i * (size_t)tiles;
    double acc = 0.0;
    for (long long m = threadIdx.x; m < tiles; m += kFinalizeThreads) acc = __dadd_rn(acc, row[m]);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1)
        acc = __dadd_rn(acc, __shfl_xor_sync(0xffffffffu, acc, off));
    if ((threadIdx.x & 31) == 0) group[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double total = group[0];
        for (int gq = 1; gq < kFinalizeThreads / 32; ++gq) total = __dadd_rn(total, group[gq]);
        loss[i] = (float)total;
    }
}

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
    if (c->flags & ~(PSOPS_KEEP_GBEST | PSOPS_QUADRATIC)) return false;
    return true;
}

Layout make_layout(const psops_config *c)
{
    Layout L{};
    const size_t kbytes = round_up(sizeof(float) * (size_t)c->K, 256);
    size_t at = 0;
    L.off_losses = at;      at += kbytes;
    L.off_pbest_loss = at;  at += kbytes;
    L.off_desc = at;        at += round_up(sizeof(SyncDesc), 256);
    L.off_gbest = at;
    if (c->flags & PSOPS_KEEP_GBEST) at += round_up(sizeof(float) * (size_t)round_up((size_t)c->N, 4), 256);
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

int launch_select(psops_ctx *ctx)
{
    const int threads = (int)round_up((size_t)ctx->cfg.K, 32);
    psops_select_kernel<<<1, threads, 0, ctx->stream>>>(ctx->loss_src, ctx->d_losses, ctx->d_pbest_loss,
                                                        ctx->d_desc, ctx->cfg.K);
    ctx->loss_src = ctx->d_losses;     // the kernel keeps a copy there
    return check_launch(ctx, "psops_select_kernel");
}

constexpr int kUnroll = PSOPS_UPDATE_UNROLL, kQuads = PSOPS_UPDATE_QUADS;
constexpr int kFitUnroll = PSOPS_FITNESS_UNROLL, kFitQuads = PSOPS_FITNESS_QUADS;
static_assert(32 % kUnroll == 0 && 32 % kFitUnroll == 0, "the improved mask is reloaded every 32 particles");
static_assert(kUpdateThreads % 32 == 0, "a warp must cover whole 128-element tiles");

template <typename Kernel>
cudaError_t launch_update_kernel(Kernel kernel, unsigned blocks, cudaStream_t stream, bool after_select,
                                 const UpdateParams &P)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(blocks, 1, 1);
    cfg.blockDim = dim3(kUpdateThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = after_select ? 1 : 0;   // overlap the launch with the selection kernel in front of it
    return cudaLaunchKernelEx(&cfg, kernel, P);
}

int launch_update(psops_ctx *ctx, float m, float k1, float k2, long long q_begin,
                  long long q_end, bool fitness, cudaStream_t stream, bool after_select = false)
{
    if (q_end <= q_begin) return PSOPS_OK;
    UpdateParams P{};
    P.x = ctx->x; P.v = ctx->v; P.p = ctx->p;
    P.gbest_copy = (ctx->cfg.flags & PSOPS_KEEP_GBEST) ? ctx->d_gbest : nullptr;
    P.dvec = ctx->dvec; P.tvec = ctx->tvec; P.partials = ctx->d_partials;
    P.desc = ctx->d_desc;
    P.ld = ctx->cfg.ld; P.N = ctx->cfg.N;
    P.q_begin = q_begin; P.q_end = q_end;
    P.tiles = ctx->tiles;
    P.K = ctx->cfg.K;
    P.m = m; P.k1 = k1; P.k2 = k2;
    fill_round_keys(ctx->cfg.seed, P.rk);
    const long long span = q_end - q_begin;
    const int per_block = kUpdateThreads * (fitness ? kFitQuads : kQuads);
    const unsigned blocks = (unsigned)((span + per_block - 1) / per_block);
    cudaError_t e;
    if (ctx->aligned) {
        if (fitness) e = launch_update_kernel(psops_update_kernel<true, true, kFitUnroll, kFitQuads>, blocks, stream, after_select, P);
        else         e = launch_update_kernel(psops_update_kernel<true, false, kUnroll, kQuads>, blocks, stream, after_select, P);
    } else {
        if (fitness) e = launch_update_kernel(psops_update_kernel<false, true, kFitUnroll, kFitQuads>, blocks, stream, after_select, P);
        else         e = launch_update_kernel(psops_update_kernel<false, false, kUnroll, kQuads>, blocks, stream, after_select, P);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "psops_update_kernel launch");
    return check_launch(ctx, "psops_update_kernel");
}

int launch_finalize(psops_ctx *ctx)
{
    psops_fitness_finalize_kernel<<<ctx->cfg.K, kFinalizeThreads, 0, ctx->stream>>>(
        ctx->d_partials, ctx->d_losses, ctx->tiles);
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
    ctx->d_gbest = (cfg->flags & PSOPS_KEEP_GBEST) ? (float *)(ctx->ws + lay.off_gbest) : nullptr;
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
    if (e == cudaSuccess) {
        // pBest_loss <- +inf (Algorithm 2 clones weights only), descriptor <- 0.
        std::vector<float> inf((size_t)cfg->K, INFINITY);
        e = cudaMemcpyAsync(ctx->d_pbest_loss, inf.data(), sizeof(float) * (size_t)cfg->K,
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
    if (ctx == nullptr || losses == nullptr) return PSOPS_EINVAL;
    const size_t bytes = sizeof(float) * (size_t)ctx->cfg.K;
    if (on_device) {
        if (((uintptr_t)losses & 3u) != 0) return PSOPS_EALIGN;
        ctx->loss_src = losses;        // read (and copied) by the selection kernel of the next sync
    } else {
        const int rc = check_host_losses(losses, ctx->cfg.K);
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
    int rc = validate_sync_args(ctx, t_iter, lambda);
    if (rc != PSOPS_OK) return rc;
    if (!ctx->have_losses) return PSOPS_ESTATE;
    const float m = inertia_of(&ctx->cfg, t_iter);
    const float k1 = ctx->cfg.c1 / lambda;
    const float k2 = ctx->cfg.c2 / lambda;
    const bool fitness = ctx->dvec != nullptr;

    rc = launch_select(ctx);
    if (rc != PSOPS_OK) return rc;
    // With the fused fitness every warp of a tile must be whole: round the
    // quad range up to a tile; quads past the end contribute +0.0.
    const long long q_end = fitness ? ctx->tiles * 32 : ctx->quads;
    rc = launch_update(ctx, m, k1, k2, 0, q_end, fitness, ctx->stream, /*after_select=*/true);
    if (rc != PSOPS_OK) return rc;
    if (fitness) {
        rc = launch_finalize(ctx);
        if (rc != PSOPS_OK) return rc;
    }
    ctx->step += 1;
    ctx->synced_once = true;
    return PSOPS_OK;
}

int psops_sync_host(psops_ctx *ctx, const float *h_x_in, int64_t h_in_ld, const float *h_losses,
                    int64_t t_iter, float lambda, float *h_x_out, int64_t h_out_ld)
{
    int rc = validate_sync_args(ctx, t_iter, lambda);
    if (rc != PSOPS_OK) return rc;
    if (h_x_in == nullptr || h_x_out == nullptr) return PSOPS_EINVAL;
    if (h_in_ld < ctx->cfg.N || h_out_ld < ctx->cfg.N) return PSOPS_EINVAL;
    rc = check_host_losses(h_losses, ctx->cfg.K);
    if (rc != PSOPS_OK) return rc;

    const int K = ctx->cfg.K;
    const long long N = ctx->cfg.N;
    const float m = inertia_of(&ctx->cfg, t_iter);
    const float k1 = ctx->cfg.c1 / lambda;
    const float k2 = ctx->cfg.c2 / lambda;
    const bool fitness = ctx->dvec != nullptr;

    if (ctx->s_in == nullptr) {
        PSOPS_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking));
        PSOPS_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking));
    }

    // Losses and selection first: the update of any element range needs them.
    PSOPS_CUDA(ctx, cudaMemcpyAsync(ctx->d_losses, h_losses, sizeof(float) * (size_t)K,
                                    cudaMemcpyHostToDevice, ctx->stream));
    ctx->loss_src = ctx->d_losses;
    ctx->have_losses = true;
    rc = launch_select(ctx);
    if (rc != PSOPS_OK) return rc;

    // Element ranges of whole tiles, about 32 MiB of weights per range.
    long long chunk_q = ((32ll << 20) / (16ll * K)) / 32 * 32;
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
    ctx->step += 1;
    ctx->synced_once = true;
    PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->s_out));
    PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return PSOPS_OK;
}

int psops_average(psops_ctx *ctx)
{
    if (ctx == nullptr) return PSOPS_EINVAL;
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
    if (ctx == nullptr) return PSOPS_EINVAL;
    if (!ctx->synced_once) return PSOPS_ESTATE;
    SyncDesc host{};
    PSOPS_CUDA(ctx, cudaMemcpyAsync(&host, ctx->d_desc, sizeof(SyncDesc), cudaMemcpyDeviceToHost, ctx->stream));
    if (pbest_loss != nullptr)
        PSOPS_CUDA(ctx, cudaMemcpyAsync(pbest_loss, ctx->d_pbest_loss, sizeof(float) * (size_t)ctx->cfg.K,
                                        cudaMemcpyDeviceToHost, ctx->stream));
    PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (g != nullptr) *g = host.g;
    if (improved_words != nullptr)
        std::memcpy(improved_words, host.improved, sizeof(uint32_t) * (size_t)((ctx->cfg.K + 31) / 32));
    return PSOPS_OK;
}

int psops_get_losses(psops_ctx *ctx, float *dst, int dst_on_device)
{
    if (ctx == nullptr || dst == nullptr) return PSOPS_EINVAL;
    if (!ctx->have_losses) return PSOPS_ESTATE;
    PSOPS_CUDA(ctx, cudaMemcpyAsync(dst, ctx->loss_src, sizeof(float) * (size_t)ctx->cfg.K,
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
    if (ctx == nullptr) return PSOPS_EINVAL;
    // The counter lives on the device (a replayed graph advances it without
    // the host taking part), so read it from there.
    SyncDesc host{};
    PSOPS_CUDA(ctx, cudaMemcpyAsync(&host, ctx->d_desc, sizeof(SyncDesc), cudaMemcpyDeviceToHost, ctx->stream));
    if (pbest_loss != nullptr)
        PSOPS_CUDA(ctx, cudaMemcpyAsync(pbest_loss, ctx->d_pbest_loss, sizeof(float) * (size_t)ctx->cfg.K,
                                        cudaMemcpyDeviceToHost, ctx->stream));
    PSOPS_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    ctx->step = host.next_step;
    if (sync_step != nullptr) *sync_step = host.next_step;
    return PSOPS_OK;
}

int psops_set_state(psops_ctx *ctx, uint32_t sync_step, const float *pbest_loss)
{
    if (ctx == nullptr || pbest_loss == nullptr) return PSOPS_EINVAL;
    for (int i = 0; i < ctx->cfg.K; ++i)
        if (pbest_loss[i] != pbest_loss[i]) return PSOPS_ENAN;
    PSOPS_CUDA(ctx, cudaMemcpyAsync(ctx->d_pbest_loss, pbest_loss, sizeof(float) * (size_t)ctx->cfg.K,
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
    if (ctx == nullptr) return PSOPS_EINVAL;
    int rc = PSOPS_OK;
    if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) rc = PSOPS_ECUDA;
    for (cudaEvent_t e : ctx->events) cudaEventDestroy(e);
    if (ctx->s_in) cudaStreamDestroy(ctx->s_in);
    if (ctx->s_out) cudaStreamDestroy(ctx->s_out);
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
    psops_fitness_finalize_kernel<<<K, kFinalizeThreads, 0, stream>>>(tile_sums, d_loss, tiles);
    if (cudaGetLastError() != cudaSuccess) return PSOPS_ECUDA;
    return PSOPS_OK;
}
