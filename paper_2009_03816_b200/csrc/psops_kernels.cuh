// psops_kernels.cuh -- device code of the PSO-PS synchronisation stage (sm_100a).
//
// Selection (Algorithm 3 + the pBest branch of Algorithm 1), the fused update
// (Eq. 6, Eq. 7), parameter averaging (Section II-B) and the quadratic
// fitness.  Included by psops.cu only; everything lives in an anonymous
// namespace.  Every floating-point operation is an explicit round-to-nearest
// intrinsic (the translation unit is built with -fmad=false, no fast-math,
// subnormals kept), so the rounding sequence is the documented one.
#pragma once

#include "psops.h"

#include <cuda_runtime.h>

#include <cstdint>

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
    int      from_kept;         // 1: gBest of this sync is the remembered row, not row g (history mode)
    float    hist_loss;         // loss of the remembered gBest (history mode)
    int      hist_valid;        // 0 until something is remembered
    unsigned int done;          // blocks of a select-in-update launch that have finished (0 between launches)
    int      pad;
    uint32_t improved[PSOPS_MAX_K / 32];   // bit i: loss_i < pBest_loss_i
};

struct UpdateParams {
    float *x, *v, *p;           // K rows of stride ld
    float *gbest_copy;          // NULL or N floats: copy of the gBest row / the remembered gBest
    const float *gbest_ext;     // NULL, or N floats holding gBest (a shard whose best particle lives elsewhere)
    const float *dvec, *tvec;   // quadratic fitness vectors (FITNESS only)
    double *partials;           // K x tiles tile sums (FITNESS only)
    const SyncDesc *desc;
    // Selection folded into this launch (SELECT): the K losses of this sync, the
    // context's copy of them, pBest_loss, and the descriptor to publish into.
    const float *loss_src;
    float *loss_keep, *pbest_loss;
    SyncDesc *desc_pub;
    long long ld, N;
    long long q_begin, q_end;   // quad range of this launch (quad = 4 elements)
    long long tiles;            // ceil(N / 128)
    int K;                      // rows held here
    int i_first;                // swarm-wide index of row 0 (0 unless the swarm is sharded by particle)
    float m, k1, k2;            // inertia, c1/lambda, c2/lambda
    uint32_t rk[20];            // Philox round keys, rk[2r], rk[2r+1]
    int group_rows;             // rows one block works on: K, or less when blockIdx.y splits the rows into groups
                                // (last on purpose: the members above keep the offsets the kernels were tuned with)
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
#define PSOPS_UPDATE_MIN_BLOCKS 0      // >0: resident blocks per SM the register allocation must allow (0: compiler's choice)
#endif
#ifndef PSOPS_FITNESS_MIN_BLOCKS
#define PSOPS_FITNESS_MIN_BLOCKS 4     // the same with the fitness fused in: 64 registers, four blocks of 256 threads
#endif
// Left to itself the compiler gives the streaming variants 80 registers (three
// blocks per SM), which is what they were tuned at; the all-resident plain
// variant it would take to 105, so that one is held at three blocks as well.
#define PSOPS_UPDATE_BOUNDS                                                          \
    __launch_bounds__(PSOPS_UPDATE_THREADS,                                          \
                      (FITNESS ? PSOPS_FITNESS_MIN_BLOCKS                            \
                               : (!SELECT && RESIDENT == 3 && U > 1) ? 3 : PSOPS_UPDATE_MIN_BLOCKS))
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
// STREAM: evict-first accesses for data far larger than L2 (every value is
// touched once per sync, so keeping it only displaces the gBest row); with
// STREAM off the accesses are ordinary write-back ones, for data that fits
// in L2 and is found there again by the next sync.  The update kernel takes
// the choice per array (x, v, pbest): see its RESIDENT parameter.
template <bool ALIGNED, bool STREAM = true>
__device__ __forceinline__ void load_quad(const float *ptr, int nvalid, float (&a)[4])
{
    if (ALIGNED && nvalid == 4) {
        const float4 t = STREAM ? __ldcs(reinterpret_cast<const float4 *>(ptr))
                                : *reinterpret_cast<const float4 *>(ptr);
        a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) a[e] = (e < nvalid) ? (STREAM ? __ldcs(ptr + e) : ptr[e]) : 0.0f;
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

template <bool ALIGNED, bool STREAM = true>
__device__ __forceinline__ void store_quad(float *ptr, int nvalid, const float (&a)[4])
{
    if (ALIGNED && nvalid == 4) {
        const float4 t = make_float4(a[0], a[1], a[2], a[3]);
        if (STREAM) __stcs(reinterpret_cast<float4 *>(ptr), t);
        else *reinterpret_cast<float4 *>(ptr) = t;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (e < nvalid) {
                if (STREAM) __stcs(ptr + e, a[e]);
                else ptr[e] = a[e];
            }
    }
}

// Level 0 of the canonical fitness sum for one quad: fp32 terms dvec*(e*e),
// widened to fp64 and added left to right.
__device__ __forceinline__ double fitness_quad_sum(const float (&xn)[4], const float (&dv)[4],
                                                   const float (&tv)[4], int nvalid)
{
    double q;
    if (nvalid == 4) {                       // every quad but the ragged last one: no per-element guards
        float term[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float err = __fsub_rn(xn[e], tv[e]);
            term[e] = __fmul_rn(dv[e], __fmul_rn(err, err));
        }
        q = __dadd_rn(__dadd_rn(__dadd_rn((double)term[0], (double)term[1]), (double)term[2]), (double)term[3]);
    } else {
        q = 0.0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            double term = 0.0;                   // elements past the end contribute +0.0
            if (e < nvalid) {
                const float err = __fsub_rn(xn[e], tv[e]);
                term = (double)__fmul_rn(dv[e], __fmul_rn(err, err));
            }
            q = (e == 0) ? term : __dadd_rn(q, term);
        }
    }
    return q;
}

// Level 1 for R rows at once (R a power of two <= 32): the xor butterfly
// a[l] += a[l ^ off], off = 16, 8, 4, 2, 1 of every row, with the rows packed
// into one register as the butterfly makes lanes redundant.  After the stage
// with offset `off` lanes l and l ^ off hold the same value, so two rows can
// share a register -- lanes with that bit clear keep the even row, lanes with
// it set take the odd row -- and the remaining stages (smaller offsets never
// cross that bit) reduce both at once.  Each row still goes through exactly
// its own butterfly tree, so the result is bit-identical to R separate
// butterflies, for R + R/2 + ... + 1 (+ what is left of the five) stages
// instead of 5 R.  On return q[0] of lane l holds the tile sum of row
// fitness_row_of_lane<R>(l).
template <int R>
__device__ __forceinline__ void fitness_tile_sums(double (&q)[R], int lane)
{
    static_assert(R >= 1 && R <= 32 && (R & (R - 1)) == 0, "rows per group must be a power of two");
#pragma unroll
    for (int s = 0; s < 5; ++s) {
        const int off = 16 >> s;
        const int n = (R >> s) > 0 ? (R >> s) : 1;       // registers still live at this stage
#pragma unroll
        for (int r = 0; r < R; ++r)
            if (r < n) q[r] = __dadd_rn(q[r], __shfl_xor_sync(0xffffffffu, q[r], off));
        if (n > 1) {
            const bool odd = (lane & off) != 0;
#pragma unroll
            for (int r = 0; r < R / 2; ++r)
                if (r < n / 2) q[r] = odd ? q[2 * r + 1] : q[2 * r];
        }
    }
}

// Row whose tile sum lane l holds after fitness_tile_sums<R>: row bit b sits in
// lane bit 4 - b.  All lanes that agree in those bits hold the same value.
template <int R>
__device__ __forceinline__ int fitness_row_of_lane(int lane)
{
    int row = 0;
#pragma unroll
    for (int b = 0; (1 << b) < R; ++b) row |= ((lane >> (4 - b)) & 1) << b;
    return row;
}

// One lane per row writes: the one whose remaining low lane bits are zero.
template <int R>
__device__ __forceinline__ bool fitness_lane_writes(int lane)
{
    return (lane & (32 / R - 1)) == 0;
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

// Arg-min over one warp's candidates: after the five stages every lane holds the winner.
__device__ __forceinline__ Candidate warp_best_candidate(Candidate c)
{
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        Candidate o;
        o.loss = __shfl_xor_sync(0xffffffffu, c.loss, off);
        o.idx = __shfl_xor_sync(0xffffffffu, c.idx, off);
        if (beats(o, c)) c = o;
    }
    return c;
}

// g_host: NULL, or a word of page-locked host memory mapped into the device's
// address space that receives g as well (particle-sharded sync: the host needs
// g to pick the rank that broadcasts its row).
__global__ void __launch_bounds__(PSOPS_MAX_K)
psops_select_kernel(const float *loss, float *loss_keep, float *__restrict__ pbest_loss,
                    SyncDesc *__restrict__ desc, int K, int history, int *g_host)
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
    c = warp_best_candidate(c);
    if (lane == 0) warp_best[warp] = c;
    __syncthreads();
    if (i == 0) {
        const int warps = (blockDim.x + 31) >> 5;
        for (int w = 1; w < warps; ++w)
            if (beats(warp_best[w], c)) c = warp_best[w];
        desc->g = c.idx;
        if (g_host != nullptr) {
            *reinterpret_cast<volatile int *>(g_host) = c.idx;
            __threadfence_system();
        }
        // Standard-PSO variant (Section II-C, step 3): gBest from the history of
        // all particles.  The current best replaces the remembered one only on
        // a strictly smaller loss, or when nothing is remembered yet.
        int from_kept = 0;
        if (history) {
            if (!desc->hist_valid || c.loss < desc->hist_loss) {
                desc->hist_loss = c.loss;
                desc->hist_valid = 1;
            } else {
                from_kept = 1;
            }
        }
        desc->from_kept = from_kept;
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
//
// SELECT (K <= 32 by construction, used up to 8; whole-range launches only): the launch does the selection
// as well, so that a sync is ONE kernel.  Every warp recomputes Algorithm 3
// and the pBest comparisons from the K losses (K L2-served floats and a
// five-stage shuffle) and then draws a ticket from an atomic counter.  The
// block that draws the LAST ticket knows that every block has read the old
// pBest_loss and step counter -- nobody reads them again in this launch -- and
// it alone publishes g, the improved mask, the new pBest_loss and the advanced
// step counter, while its own row loads are in flight.  No block ever waits
// for another.
//
// RESIDENT = how many of the arrays x, v, pbest (in that order) are accessed
// with ordinary write-back loads and stores; the rest is streamed evict-first.
// 0 for a swarm far larger than L2; 3 for one that fits; 1 or 2 in between:
// the streamed arrays then pass through L2 without displacing the resident
// ones, which the next sync finds there (x and v are read AND written each
// sync, pbest only one of the two, hence the order).
// ---------------------------------------------------------------------------
template <bool ALIGNED, bool FITNESS, bool SELECT, int RESIDENT, int U, int Q, bool SPLIT = false>
__global__ void PSOPS_UPDATE_BOUNDS
psops_update_kernel(const __grid_constant__ UpdateParams P)
{
    static_assert(!(SELECT && FITNESS), "the single-launch form carries no fitness");
    static_assert(RESIDENT >= 0 && RESIDENT <= 3, "x, v, pbest");
    constexpr bool STREAM_X = RESIDENT < 1, STREAM_V = RESIDENT < 2, STREAM_P = RESIDENT < 3;
    const long long q0 = P.q_begin + (long long)blockIdx.x * (kUpdateThreads * Q) + threadIdx.x;
    // Whatever follows in the stream with programmatic serialisation (the
    // fitness finaliser, the next sync) may be made resident now; it waits for
    // this grid to finish before it reads anything.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Launched with programmatic stream serialisation behind the kernel in
    // front of it: everything that kernel wrote is visible after this wait (a
    // no-op for an ordinary launch).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!FITNESS && !SELECT && q0 >= P.q_end) return;   // with FITNESS whole warps stay for the shuffles,
                                                        // with SELECT whole blocks for the barrier below

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
    const int lane = threadIdx.x & 31;

    // Rows this block works on: all K of them, or -- for a swarm of many
    // particles and few elements, which would otherwise leave most SMs idle
    // while each thread walks all K rows -- the group blockIdx.y picks.  A
    // launch that splits the rows is always given gBest in a buffer of its own
    // (P.gbest_ext): the block that overwrites row g is then no longer the only
    // one that reads it.
    // SPLIT is a compile-time switch so that the ordinary launches carry none of
    // it: their row count is written as the kernel parameter itself below (a
    // local copy of it cost the one-particle-in-flight variant 15 %).
    const int k0 = SPLIT ? (int)blockIdx.y * P.group_rows : 0;
    const int Kg = (P.K - k0 < P.group_rows) ? P.K - k0 : P.group_rows;   // used with SPLIT only
    const int ifirst = P.i_first + k0;       // swarm-wide index of this block's first row
#define PSOPS_ROWS (SPLIT ? Kg : P.K)

    // Selection results: read from the descriptor the selection kernel filled,
    // or (SELECT) recomputed here by every warp; lane i stands for particle i.
    uint32_t step;
    int g;
    int from_kept = 0;
    uint32_t sel_word = 0;                   // SELECT: improved bits of particles 0..31
    float sel_loss = 0.0f;
    bool sel_improved = false;
    if (SELECT) {
        const bool live = lane < P.K;
        sel_loss = live ? __ldcg(P.loss_src + lane) : 0.0f;
        const float pl = live ? __ldcg(P.pbest_loss + lane) : 0.0f;
        sel_improved = live && (sel_loss < pl);          // strict: an equal loss never replaces pBest
        sel_word = __ballot_sync(0xffffffffu, sel_improved);
        Candidate c;
        c.loss = live ? sel_loss : __int_as_float(0x7fc00000);
        c.idx = live ? lane : 0x7fffffff;
        g = warp_best_candidate(c).idx;
        step = __ldcg(&P.desc_pub->next_step);
        // g and the ballot needed every lane's loads: past this barrier all warps
        // of the block hold the old selection state in registers, and the block's
        // ticket (drawn below, under the first row loads) may say so.
        __syncthreads();
    } else {
        step = P.desc->step;
        g = P.desc->g;
        from_kept = P.desc->from_kept;
    }

    // gBest = row g as it is BEFORE this sync overwrites it; this thread is the
    // only writer of these elements, so reading them first is enough.
    // It comes from row g of this context, from the remembered row (history
    // mode, when the current best did not beat it) or from a row handed in by
    // the caller (sharded swarm).
    const float *gsrc = P.gbest_ext;
    bool keep_copy = P.gbest_copy != nullptr;
    if (gsrc == nullptr) {
        if (from_kept) {
            gsrc = P.gbest_copy;
            keep_copy = false;               // it is the copy
        } else {
            gsrc = P.x + (size_t)g * (size_t)P.ld;
        }
    }
    float gb[Q][4];
    float dv[Q][4], tv[Q][4];
#pragma unroll
    for (int j = 0; j < Q; ++j) {
        load_quad_cached<ALIGNED>(gsrc + col[j], nvalid[j], gb[j]);
        if (keep_copy) store_quad<ALIGNED, STREAM_X>(P.gbest_copy + col[j], nvalid[j], gb[j]);
        if (FITNESS) {
            load_quad_cached<ALIGNED>(P.dvec + col[j], nvalid[j], dv[j]);
            load_quad_cached<ALIGNED>(P.tvec + col[j], nvalid[j], tv[j]);
        }
    }

    // Philox counter word 0 = element >> 1: 2q for elements 4q, 4q+1 and
    // 2q + 1 for elements 4q+2, 4q+3.
    const uint32_t pair0 = (uint32_t)(2 * q0);

    // With the fitness fused in, the warp reduction of a batch is carried into
    // the next iteration and runs right after that iteration's loads have been
    // issued, so that the shuffle chain sits in the shadow of the loads.
    double fq[Q][U];                         // level-0 fitness sums of the previous batch
    int fq_i0 = -1;
    auto flush_fitness = [&]() {
#pragma unroll
        for (int j = 0; j < Q; ++j) {
            fitness_tile_sums<U>(fq[j], lane);
            const int i = fq_i0 + fitness_row_of_lane<U>(lane);
            if (fitness_lane_writes<U>(lane) && active[j] && i < PSOPS_ROWS)    // q_end is a whole number of tiles
                P.partials[(size_t)(k0 + i) * (size_t)P.tiles + (col[j] >> 7)] = fq[j][0];
        }
    };

    size_t row = (size_t)k0 * (size_t)P.ld;  // offset of row i0 of this block's group
    uint32_t impw = sel_word;                // improved bits of particles i0 - i0 % 32 .. +31 (the group's numbering)
    for (int i0 = 0; i0 < PSOPS_ROWS; i0 += U) {
        if (!SELECT && (i0 & 31) == 0) {
            // One window of 32 bits per 32 particles, fetched ahead of the loads it
            // steers: a per-particle fetch would sit between them and stall the
            // in-order issue.  The window starts at swarm-wide particle i_first + i0.
            const int base = ifirst + i0;
            const uint32_t lo = P.desc->improved[base >> 5];
            const uint32_t hi = ((base >> 5) + 1 < PSOPS_MAX_K / 32) ? P.desc->improved[(base >> 5) + 1] : 0u;
            impw = __funnelshift_r(lo, hi, base & 31);
        }

        float xo[U][Q][4], vo[U][Q][4], pp[U][Q][4];
        bool imp[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + u;
            imp[u] = (impw >> (i & 31)) & 1u;
            if (i < PSOPS_ROWS) {
#pragma unroll
                for (int j = 0; j < Q; ++j) {
                    const size_t at = row + (size_t)u * (size_t)P.ld + col[j];
                    load_quad<ALIGNED, STREAM_X>(P.x + at, nvalid[j], xo[u][j]);
                    load_quad<ALIGNED, STREAM_V>(P.v + at, nvalid[j], vo[u][j]);
                    if (!imp[u]) load_quad<ALIGNED, STREAM_P>(P.p + at, nvalid[j], pp[u][j]);
                }
            }
        }
        if (SELECT && i0 == 0 && threadIdx.x < 32) {
            // The ticket, in the shadow of the loads just issued.  Whoever draws the
            // last one publishes; the others carry on at once.
            unsigned int ticket = 0;
            if (lane == 0) ticket = atomicAdd(&P.desc_pub->done, 1u);
            ticket = __shfl_sync(0xffffffffu, ticket, 0);
            if (ticket == gridDim.x - 1) {
                if (lane < P.K) {
                    P.loss_keep[lane] = sel_loss;                 // the context's own copy of the losses
                    if (sel_improved) P.pbest_loss[lane] = sel_loss;
                }
                if (lane == 0) {
                    SyncDesc *d = P.desc_pub;
                    d->g = g;
                    d->improved[0] = sel_word;
                    d->from_kept = 0;
                    d->step = step;
                    d->next_step = step + 1u;
                    d->done = 0u;                                 // every ticket of this launch has been drawn
                }
            }
        }
        if (FITNESS) {
            if (fq_i0 >= 0) flush_fitness();     // previous batch, under this batch's loads
#pragma unroll
            for (int j = 0; j < Q; ++j)
#pragma unroll
                for (int u = 0; u < U; ++u) fq[j][u] = 0.0;   // rows past K carry +0.0 and are not written
            fq_i0 = i0;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + u;
            if (i < PSOPS_ROWS) {
#pragma unroll
                for (int j = 0; j < Q; ++j) {
                    const size_t at = row + (size_t)u * (size_t)P.ld + col[j];
                    const uint32_t pair = pair0 + (uint32_t)(2 * j * kUpdateThreads);
                    uint32_t ra[4], rb[4];
                    philox4x32_10(pair, (uint32_t)(ifirst + i), step, 0u, P.rk, ra);
                    philox4x32_10(pair + 1u, (uint32_t)(ifirst + i), step, 0u, P.rk, rb);
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
                    store_quad<ALIGNED, STREAM_V>(P.v + at, nvalid[j], vn);
                    store_quad<ALIGNED, STREAM_X>(P.x + at, nvalid[j], xn);
                    if (imp[u]) store_quad<ALIGNED, STREAM_P>(P.p + at, nvalid[j], xo[u][j]);
                    if (FITNESS) fq[j][u] = fitness_quad_sum(xn, dv[j], tv[j], nvalid[j]);
                }
            }
        }
        row += (size_t)U * (size_t)P.ld;
    }
    if (FITNESS && fq_i0 >= 0) flush_fitness();
#undef PSOPS_ROWS
}

// ---------------------------------------------------------------------------
// gBest snapshot for launches of kernel (b) that split the rows over
// blockIdx.y: row g of x, as the selection kernel in front of it chose it, is
// copied to `dst` before the update overwrites it.
// ---------------------------------------------------------------------------
template <bool ALIGNED>
__global__ void __launch_bounds__(kUpdateThreads)
psops_gbest_snapshot_kernel(const SyncDesc *__restrict__ desc, const float *__restrict__ x, long long ld,
                            long long N, long long quads, float *__restrict__ dst)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");         // the selection kernel has written desc->g
    const long long q = (long long)blockIdx.x * kUpdateThreads + threadIdx.x;
    if (q >= quads) return;
    const long long d0 = q * 4;
    const int nvalid = (N - d0 >= 4) ? 4 : (int)(N - d0);
    float a[4];
    load_quad_cached<ALIGNED>(x + (size_t)desc->g * (size_t)ld + d0, nvalid, a);
    store_quad<ALIGNED, false>(dst + d0, nvalid, a);
}

// The same snapshot with the selection folded in (K <= 32): every warp
// recomputes Algorithm 3 and the pBest comparisons as in the single-launch
// form of kernel (b), each thread copies its quad of row g, and the block that
// draws the last ticket publishes the selection for the update kernel behind
// it.  One launch instead of two in front of a row-split update.
template <bool ALIGNED>
__global__ void __launch_bounds__(kUpdateThreads)
psops_select_snapshot_kernel(const float *loss_src, float *loss_keep, float *pbest_loss, SyncDesc *desc, int K,
                             const float *__restrict__ x, long long ld, long long N, long long quads,
                             float *__restrict__ dst)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31;
    const bool live = lane < K;
    const float li = live ? __ldcg(loss_src + lane) : 0.0f;
    const float pl = live ? __ldcg(pbest_loss + lane) : 0.0f;
    const bool improved = live && (li < pl);                 // strict: an equal loss never replaces pBest
    const uint32_t word = __ballot_sync(0xffffffffu, improved);
    Candidate c;
    c.loss = live ? li : __int_as_float(0x7fc00000);
    c.idx = live ? lane : 0x7fffffff;
    const int g = warp_best_candidate(c).idx;
    const uint32_t step = __ldcg(&desc->next_step);
    __syncthreads();                                         // all warps of the block hold the old state in registers

    const long long q = (long long)blockIdx.x * kUpdateThreads + threadIdx.x;
    const long long d0 = q * 4;
    const int nvalid = (q < quads) ? ((N - d0 >= 4) ? 4 : (int)(N - d0)) : 0;
    float a[4];
    load_quad_cached<ALIGNED>(x + (size_t)g * (size_t)ld + d0, nvalid, a);
    if (threadIdx.x < 32) {                                  // the ticket, under the load just issued
        unsigned int ticket = 0;
        if (lane == 0) ticket = atomicAdd(&desc->done, 1u);
        ticket = __shfl_sync(0xffffffffu, ticket, 0);
        if (ticket == gridDim.x - 1) {                       // every block has read the old state: move it on
            if (live) {
                loss_keep[lane] = li;
                if (improved) pbest_loss[lane] = li;
            }
            if (lane == 0) {
                desc->g = g;
                desc->improved[0] = word;
                desc->from_kept = 0;
                desc->step = step;
                desc->next_step = step + 1u;
                desc->done = 0u;
            }
        }
    }
    store_quad<ALIGNED, false>(dst + d0, nvalid, a);
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
// Synchronous SGD (Section II-B): w <- w + (alpha / K) sum_k grad_k, written to
// every worker's row; the new weight is computed from row 0.
// ---------------------------------------------------------------------------
template <bool ALIGNED, int U>
__global__ void __launch_bounds__(kUpdateThreads)
psops_ssgd_kernel(float *__restrict__ w, const float *__restrict__ grad, long long ld, long long grad_ld,
                  long long N, long long quads, int K, float scale)
{
    const long long q = (long long)blockIdx.x * kUpdateThreads + threadIdx.x;
    if (q >= quads) return;
    const long long d0 = q * 4;
    const int nvalid = (N - d0 >= 4) ? 4 : (int)(N - d0);

    float w0[4], acc[4];
    load_quad<ALIGNED>(w + d0, nvalid, w0);
    load_quad<ALIGNED>(grad + d0, nvalid, acc);
    for (int k = 1; k < K; k += U) {
        float t[U][4];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (k + u < K) load_quad<ALIGNED>(grad + (size_t)(k + u) * (size_t)grad_ld + d0, nvalid, t[u]);
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (k + u < K) {
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[e] = __fadd_rn(acc[e], t[u][e]);
            }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) w0[e] = __fadd_rn(w0[e], __fmul_rn(scale, acc[e]));
    for (int k = 0; k < K; ++k) store_quad<ALIGNED>(w + (size_t)k * (size_t)ld + d0, nvalid, w0);
}

// ---------------------------------------------------------------------------
// Kernel (d): stand-alone fitness tile sums (levels 0 and 1), and the level-2
// finalisation shared with the fused path.
// ---------------------------------------------------------------------------
#ifndef PSOPS_FITNESS_ROWS
#define PSOPS_FITNESS_ROWS 4           // rows per group in the stand-alone fitness kernel (power of two)
#endif
template <bool ALIGNED>
__global__ void __launch_bounds__(kUpdateThreads)
psops_fitness_tiles_kernel(const float *__restrict__ x, const float *__restrict__ dvec,
                           const float *__restrict__ tvec, double *__restrict__ partials,
                           long long ld, long long N, long long quads, long long tiles, int K)
{
    const long long q = (long long)blockIdx.x * kUpdateThreads + threadIdx.x;
    const long long d0 = q * 4;
    int nvalid = 0;
    // the finaliser behind this kernel may be made resident; it waits for this grid
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (q < quads) nvalid = (N - d0 >= 4) ? 4 : (int)(N - d0);
    if ((q >> 5) >= tiles) return;           // whole warp out of range
    float dv[4], tv[4];
    load_quad_cached<ALIGNED>(dvec + d0, nvalid, dv);
    load_quad_cached<ALIGNED>(tvec + d0, nvalid, tv);
    constexpr int U = PSOPS_FITNESS_ROWS;    // rows in flight per thread
    for (int i0 = 0; i0 < K; i0 += U) {
        float xi[U][4];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (i0 + u < K) load_quad<ALIGNED>(x + (size_t)(i0 + u) * (size_t)ld + d0, nvalid, xi[u]);
        double fq[U];
#pragma unroll
        for (int u = 0; u < U; ++u) fq[u] = (i0 + u < K) ? fitness_quad_sum(xi[u], dv, tv, nvalid) : 0.0;
        const int lane = threadIdx.x & 31;
        fitness_tile_sums<U>(fq, lane);
        const int i = i0 + fitness_row_of_lane<U>(lane);
        if (fitness_lane_writes<U>(lane) && i < K)
            partials[(size_t)i * (size_t)tiles + (size_t)(q >> 5)] = fq[0];
    }
}

// Level 2.  The 1024 slots of one particle are spread over a cluster of 8
// thread blocks (128 slots = 4 groups of 32 each), so eight SMs stream the
// particle's tile sums instead of one; thread tau still adds tiles tau,
// tau + 1024, ... in increasing order (loads run ahead, the additions stay a
// chain), each warp butterflies its group, and the 32 group sums meet in the
// shared memory of the cluster's first block, whose first thread adds them in
// group order.  cluster.sync() is the hardware cluster barrier; the
// arrive/wait pair in front of the remote store is the same barrier, split so
// that the wait comes after the loads.
#ifndef PSOPS_FINALIZE_DEPTH
#define PSOPS_FINALIZE_DEPTH 32        // tile sums in flight per thread of the finaliser
#endif
constexpr int kFinalizeCluster = 8;
constexpr int kFinalizeCtaThreads = kFinalizeThreads / kFinalizeCluster;
static_assert(kFinalizeCtaThreads % 32 == 0, "a warp is one group of 32 slots");

__global__ void __cluster_dims__(kFinalizeCluster, 1, 1) __launch_bounds__(kFinalizeCtaThreads)
psops_fitness_finalize_kernel(const double *__restrict__ partials, float *__restrict__ loss,
                              long long tiles)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ double group[kFinalizeThreads / 32];
    const unsigned rank = cluster.block_rank();
    const int i = blockIdx.y;
    const int tau = (int)rank * kFinalizeCtaThreads + (int)threadIdx.x;      // slot
    const double *row = partials + (size_t)i * (size_t)tiles;
    // Another block's shared memory may only be touched once that block is
    // running: every block arrives at the cluster barrier here and waits for
    // the others just before the remote store, after its own loads.
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    // Launched with programmatic stream serialisation behind the kernel that
    // writes the tile sums: they are visible after this wait.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    double acc = 0.0;
    // Only 1024 chains per particle exist, so each thread keeps many loads in
    // flight; the volatile asm keeps the compiler from trading them for registers.
    constexpr int D = PSOPS_FINALIZE_DEPTH;
    long long m = tau;
    for (; m + (long long)(D - 1) * kFinalizeThreads < tiles; m += (long long)D * kFinalizeThreads) {
        double v[D];
#pragma unroll
        for (int d = 0; d < D; ++d)
            asm volatile("ld.global.f64 %0, [%1];" : "=d"(v[d]) : "l"(row + m + (long long)d * kFinalizeThreads));
#pragma unroll
        for (int d = 0; d < D; ++d) acc = __dadd_rn(acc, v[d]);
    }
    {
        // The last, partial batch the same way -- loads first, then the chain of
        // additions -- so that it costs one memory latency and not one per tile.
        double v[D];
#pragma unroll
        for (int d = 0; d < D; ++d) {
            v[d] = 0.0;
            if (m + (long long)d * kFinalizeThreads < tiles)
                asm volatile("ld.global.f64 %0, [%1];" : "=d"(v[d]) : "l"(row + m + (long long)d * kFinalizeThreads));
        }
#pragma unroll
        for (int d = 0; d < D; ++d)
            if (m + (long long)d * kFinalizeThreads < tiles) acc = __dadd_rn(acc, v[d]);
    }

#pragma unroll
    for (int off = 16; off >= 1; off >>= 1)
        acc = __dadd_rn(acc, __shfl_xor_sync(0xffffffffu, acc, off));
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");      // all blocks of the cluster run
    if ((threadIdx.x & 31) == 0) {
        double *first = cluster.map_shared_rank(group, 0);
        first[tau >> 5] = acc;
    }
    cluster.sync();
    if (rank == 0 && threadIdx.x == 0) {
        double total = group[0];
        for (int gq = 1; gq < kFinalizeThreads / 32; ++gq) total = __dadd_rn(total, group[gq]);
        loss[i] = (float)total;
    }
}

} // namespace
