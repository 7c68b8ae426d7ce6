/*
 * psops.h -- C ABI of the B200 PSO-PS parameter-synchronisation library.
 *
 * PSO-PS (Ye, Han, Sun, Lv, "PSO-PS: Parameter Synchronization with Particle
 * Swarm Optimization for Distributed Training of Deep Neural Networks")
 * replaces the averaging step of data-parallel training by a particle-swarm
 * update: the K workers' weight vectors are particles (Table I: position =
 * weights, fitness = training loss), each with a velocity and a personal best,
 * and at every synchronisation point new weights come from Eq. 6 / Eq. 7
 * instead of from the mean.  This library is that synchronisation stage for K
 * particles held as K flat fp32 rows in one GPU's memory.
 *
 * Conventions
 *   - All entry points return 0 (PSOPS_OK) or a negative PSOPS_E* code; none
 *     throws, aborts or prints.  Arguments are validated before any launch.
 *   - "device pointer" = address in the memory of the GPU that was current
 *     when psops_create ran; "host pointer" = ordinary process memory.
 *   - The library allocates no device memory.  The caller owns x, v, pbest,
 *     the workspace, dvec/tvec and the stream, and keeps them alive until
 *     psops_destroy.  The context itself is host memory owned by the library.
 *   - A context belongs to the GPU that was current in psops_create; later
 *     calls switch to that GPU for their duration if another one is current.
 *   - A context is not thread-safe: one host thread at a time per context.
 *     Different contexts are independent (different streams run concurrently).
 *   - Work is enqueued on the stream given at creation.  Calls that fill a
 *     host buffer wait for that stream before they return; the others do not.
 *   - Rows: particle i occupies elements [i*ld, i*ld + N) of x, v and pbest.
 *     Elements [N, ld) of a row are padding and are never written.
 *     If x, v, pbest are 16-byte aligned and ld % 4 == 0 the 128-bit kernels
 *     run; otherwise a scalar variant with identical results runs.
 *   - Random numbers: r1, r2 of Eq. 6 are drawn per (particle, element, sync)
 *     from Philox4x32-10 with counter {element >> 1, particle, sync step, 0}
 *     and key {seed low word, seed high word}; the even element of a pair
 *     takes output words 0,1 and the odd element words 2,3; a word w becomes
 *     (w >> 8) * 2^-24 in [0, 1).  The stream is a pure function of those
 *     indices, so a context has no generator state beyond its step counter.
 */
#ifndef PSOPS_H
#define PSOPS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PSOPS_OK           0
#define PSOPS_EINVAL      -1   /* null pointer, size or hyper-parameter out of range   */
#define PSOPS_EALIGN      -2   /* a device pointer is not 4-byte aligned               */
#define PSOPS_ESTATE      -3   /* call order: e.g. sync before any losses were given   */
#define PSOPS_ENAN        -4   /* a host-supplied loss is NaN                          */
#define PSOPS_EWORKSPACE  -5   /* workspace missing, misaligned (256 B) or too small   */
#define PSOPS_ECUDA       -6   /* a CUDA call failed; psops_last_error has its text    */
#define PSOPS_ENOMEM      -7   /* host allocation of the context failed                */
#define PSOPS_ELIMIT      -8   /* size beyond the built-in scratch (psops_quadratic_fitness_static) */

#define PSOPS_MAX_K     1024

/* psops_config.flags */
#define PSOPS_KEEP_GBEST   1u  /* keep a copy of the gBest row of each sync (+4N bytes of workspace) */
#define PSOPS_QUADRATIC    2u  /* reserve workspace for the on-device quadratic fitness              */
#define PSOPS_GBEST_HISTORY 4u /* gBest = best of all syncs so far instead of this sync's best (+4N bytes) */
#define PSOPS_SEPARATE_SELECT 8u /* always run the selection as a kernel of its own (see psops_sync)       */

/* `which` of psops_get_weights / psops_set_weights */
#define PSOPS_X      0         /* weights  w_i  (position of particle i)     */
#define PSOPS_V      1         /* velocity v_i                               */
#define PSOPS_PBEST  2         /* personal best pBest_i                      */
#define PSOPS_GBEST  3         /* gBest of the last sync (needs KEEP_GBEST)  */

typedef struct psops_ctx psops_ctx;      /* opaque */

/* Hyper-parameters (Table II) and geometry of one swarm. */
typedef struct {
    int32_t  K;              /* particles = workers (Table I) held by this context, 1..PSOPS_MAX_K */
    int32_t  k_first;        /* swarm-wide index of row 0; 0 unless the swarm is sharded    */
    int64_t  N;              /* elements per particle, 1 .. 2^33 - 1                        */
    int64_t  ld;             /* row stride in elements, ld >= N                             */
    float    m_max, m_min;   /* Eq. 5; m_max == m_min gives a constant inertia weight       */
    int64_t  t_max;          /* Eq. 5 denominator (Max_t of Algorithm 1), >= 1              */
    float    c1, c2;         /* acceleration constants of Eq. 6                             */
    uint64_t seed;           /* Philox key                                                  */
    uint32_t flags;          /* PSOPS_KEEP_GBEST | PSOPS_QUADRATIC | PSOPS_GBEST_HISTORY |
                                PSOPS_SEPARATE_SELECT                                       */
    int32_t  K_total;        /* particles in the whole swarm when this context holds a shard
                                [k_first, k_first + K) of it; 0 = not sharded (K_total = K)  */
} psops_config;

/* Bytes of device workspace a context with this configuration needs
 * (0 if the configuration is invalid).  The workspace must be 256-byte
 * aligned. */
size_t psops_workspace_bytes(const psops_config *cfg);

/*
 * Particle initialisation (Algorithm 2): adopt the caller's device rows as the
 * swarm.  d_x, d_v, d_pbest: K rows of stride ld each, fp32, already holding
 * the initial weights, velocities and personal bests (Algorithm 2 clones the
 * weights, so callers normally pass pbest == a copy of x).  pBest_loss starts
 * at +inf (the paper initialises no loss), the sync counter at 0.
 * cuda_stream: a cudaStream_t (NULL = the legacy default stream).
 * Errors: EINVAL, EALIGN, EWORKSPACE, ENOMEM, ECUDA.  On error *out is NULL.
 */
int psops_create(psops_ctx **out, const psops_config *cfg,
                 float *d_x, float *d_v, float *d_pbest,
                 void *d_workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Hand in the current training losses of the whole swarm (the fitness of
 * Table I; lower is better): K floats, K_total on a shard.  on_device == 0: host pointer, checked for NaN (ENAN) and copied
 * before the call returns to the stream (the buffer may be reused at once).
 * on_device != 0: device pointer (4-byte aligned), not inspected and not
 * copied now: the selection kernel of the next psops_sync reads it on the
 * stream (and keeps a copy), so the buffer must stay valid and unchanged until
 * that sync has run.
 */
int psops_set_losses(psops_ctx *ctx, const float *losses, int on_device);

/*
 * One synchronisation: the "t % step == 0" branch of Algorithm 1.
 *   1. gBest = weights of the particle with the smallest loss at this
 *      iteration (Algorithm 3); ties go to the lowest particle index; a NaN
 *      loss never beats a number.
 *   2. every particle with loss_i < pBest_loss_i (strict) sets pBest_i to its
 *      current weights and pBest_loss_i to loss_i.
 *   3. v_i <- m v_i + (c1 r1/lambda)(pBest_i - w_i) + (c2 r2/lambda)(gBest - w_i)
 *      (Eq. 6) and w_i <- w_i + v_i (Eq. 7), with m from Eq. 5 at iteration
 *      t_iter (clamped to t_max).  Rounding sequence per element, all fp32
 *      round-to-nearest: dl = pBest - w; dg = gBest - w; t1 = (c1/lambda) r1;
 *      t2 = (c2/lambda) r2; a0 = m v; v' = fma(t2, dg, fma(t1, dl, a0));
 *      w' = w + v'.
 * If a quadratic fitness is attached (psops_set_quadratic) the losses of the
 * NEW weights are evaluated in the same pass and become the losses of the next
 * sync.  Enqueues work only; the sync counter advances by one.  The counter
 * lives in device memory and is advanced by the selection kernel itself, so a
 * psops_sync recorded into a CUDA graph (with the losses in a device buffer,
 * see psops_set_losses) keeps walking the random stream when the graph is
 * replayed; t_iter and lambda are then the ones given at capture.
 * Launches: a small swarm -- at most 8 particles, no history variant, no fused
 * fitness, and few enough elements that all thread blocks of the update are
 * resident at once (on a B200 about 450,000 with up to 4 particles, 150,000
 * with 5 to 8) -- is launch-bound, and its whole sync is ONE kernel: every
 * thread block recomputes steps 1 and 2 from the K losses, and the block that
 * draws the last ticket of a counter publishes g, the improved mask, pBest_loss
 * and the counter (no block waits for another).  Otherwise, or with
 * PSOPS_SEPARATE_SELECT, a selection kernel runs first and the update kernel
 * behind it.  A swarm of 9 or more particles on few elements (up to 2^19, and
 * few enough that one block column per 1024 elements would leave SMs idle) has
 * its rows split into groups that run side by side; since row g is then read
 * by blocks that do not write it, a small kernel first copies it into the
 * workspace -- up to 32 particles that kernel also does the selection (two
 * launches per sync), beyond 32 or with PSOPS_SEPARATE_SELECT the selection
 * kernel runs in front of it (three).  The results are identical bit for bit in
 * every form.
 * Cache policy: of the arrays x, v, pbest (4 K N bytes each) as many as fit
 * together in about half of the GPU's L2 cache are accessed with ordinary
 * loads and stores, so that the next sync finds them there; the others, and
 * everything in a swarm far larger than L2, are streamed (evict-first).
 * Errors: EINVAL (t_iter < 0, lambda < 1 or not finite), ESTATE (no losses
 * yet), ECUDA.
 */
int psops_sync(psops_ctx *ctx, int64_t t_iter, float lambda);

/*
 * Same synchronisation for callers whose weights live in host memory (the
 * workers' side of Algorithm 1: gather weights and losses, distribute new
 * weights).  h_x_in: K rows of stride h_in_ld (>= N) with the workers' current
 * weights; h_losses: K losses; h_x_out: K rows of stride h_out_ld receiving
 * the new weights (may equal h_x_in).  Velocities and personal bests stay on
 * the device.  Copies and kernels are pipelined over element ranges; the call
 * returns when h_x_out is complete.  Pinned host memory gives full speed.
 * Errors: as psops_sync, plus ENAN.  Also on an error from the CUDA runtime the
 * call returns only after every copy and kernel it had queued has finished, so
 * the host buffers may be freed at once; the swarm's state is then undefined
 * (some element ranges updated, others not).
 */
int psops_sync_host(psops_ctx *ctx, const float *h_x_in, int64_t h_in_ld,
                    const float *h_losses, int64_t t_iter, float lambda,
                    float *h_x_out, int64_t h_out_ld);

/*
 * Page-lock (pin) a host buffer that psops_sync_host will use, and release it
 * again.  With ordinary pageable memory the copies of psops_sync_host are
 * staged by the driver and run several times slower (measured: 6x); pin the
 * buffers once, reuse them for every sync, unregister before freeing them.
 * Registering an already registered range is not an error.  EINVAL, ECUDA.
 */
int psops_host_register(void *host_ptr, size_t bytes);
int psops_host_unregister(void *host_ptr);

/*
 * Particle-sharded synchronisation: each GPU holds K of the swarm's K_total
 * particles (psops_config.k_first / K_total) and only the best particle's
 * weights travel -- the exchange Algorithm 3 describes as a gather of all
 * particles reduces to an all-gather of K_total losses plus one broadcast of N
 * floats.  Per sync, on every shard:
 *   1. psops_set_losses with all K_total losses (the caller's all-gather);
 *   2. psops_shard_select: Algorithm 3 and the pBest branch over the whole
 *      swarm; *g receives the swarm-wide gBest index (waits for the stream);
 *   3. the shard that holds particle g copies that row out (psops_get_weights)
 *      and the caller broadcasts it into a buffer in every GPU's own memory;
 *   4. psops_shard_update: Eq. 6 / Eq. 7 for this shard's particles with gBest
 *      read from d_gbest_row (N floats, device pointer, 16-byte aligned on the
 *      128-bit path).  Random draws use the swarm-wide particle index, so the
 *      result is that of one unsharded psops_sync.  The shard that holds
 *      particle g may pass that row of its own x directly: every element of
 *      gBest is read by the thread that later overwrites it.
 *      psops_shard_update_range does step 4 for elements [first_elem,
 *      last_elem) only, so that the broadcast can travel in pieces and the
 *      update of one piece runs while the next is still on the wire: call it
 *      with consecutive ranges from 0 to N (first_elem a multiple of 4,
 *      last_elem a multiple of 4 or N; d_gbest_row always points at element 0 of
 *      the row, of which only the range is read); the sync counter advances when
 *      the range that ends at N has been enqueued.
 * psops_shard_select waits only for the selection kernel (an event behind it;
 * g arrives through a page-locked word the kernel writes), not for later work.
 * psops_sync, psops_sync_host, psops_average and psops_ssgd return ESTATE on a
 * sharded context (they need the whole swarm).  The quadratic fitness and
 * PSOPS_GBEST_HISTORY are not available on shards; PSOPS_KEEP_GBEST is (the
 * shard keeps a copy of the row it was given).
 * Errors: EINVAL, EALIGN, ESTATE (no losses / update without select / a second
 * select before the update is complete / a range out of order), ECUDA.
 */
int psops_shard_select(psops_ctx *ctx, int *g);
int psops_shard_update(psops_ctx *ctx, int64_t t_iter, float lambda, const float *d_gbest_row);
int psops_shard_update_range(psops_ctx *ctx, int64_t t_iter, float lambda, const float *d_gbest_row,
                             int64_t first_elem, int64_t last_elem);

/*
 * gBest from the history of all particles (the standard-PSO framework of
 * Section II-C, step 3, in place of Algorithm 3's best-of-this-iteration):
 * with PSOPS_GBEST_HISTORY the context remembers the best row ever selected
 * and its loss; a sync's arg-min particle replaces it only on a strictly
 * smaller loss (or when nothing is remembered yet), and Eq. 6 uses the
 * remembered row.  psops_get_weights(PSOPS_GBEST) returns that row.  These two
 * calls move the remembered loss (and, for set, the row) for checkpoint/resume.
 */
int psops_get_history(psops_ctx *ctx, float *gbest_loss, int *valid);
int psops_set_history(psops_ctx *ctx, float gbest_loss, const float *gbest_row, int row_on_device);

/*
 * Synchronous SGD as the paper states it beside parameter averaging
 * (Section II-B): w <- w + (alpha / K) sum_k grad_k, written to every row of x
 * (the new weight is computed from row 0).  d_grad: K rows of stride grad_ld
 * (>= N), device pointer.  fp32: gradients summed in worker order, one division
 * alpha / K, one product, one addition.  v, pbest and the sync counter are
 * untouched.
 */
int psops_ssgd(psops_ctx *ctx, const float *d_grad, int64_t grad_ld, float alpha);

/*
 * Parameter averaging, the baseline the paper compares with (Section II-B,
 * step 5): every w_i <- (1/K) sum_k w_k.  fp32 sum in particle order, one
 * division.  Velocities, personal bests and the sync counter are untouched.
 */
int psops_average(psops_ctx *ctx);

/*
 * Copy one row out.  which = PSOPS_X / PSOPS_V / PSOPS_PBEST with particle k in
 * [0, K), or PSOPS_GBEST (k ignored): the gBest row used by the last sync,
 * available only with PSOPS_KEEP_GBEST (else ESTATE, as the pre-update row no
 * longer exists).  dst receives N floats; dst_on_device selects the kind of
 * pointer; a host destination is complete on return.
 */
int psops_get_weights(psops_ctx *ctx, int which, int k, float *dst, int dst_on_device);

/* Overwrite row k of x, v or pbest with N floats from src (host or device). */
int psops_set_weights(psops_ctx *ctx, int which, int k, const float *src, int src_on_device);

/*
 * Selection results of the last sync, copied to host memory (each pointer may
 * be NULL): *g = gBest index; improved_words[(K+31)/32], bit i set when
 * particle i improved; pbest_loss[K] after the update.  Waits for the stream.
 * ESTATE before the first sync.
 */
int psops_sync_info(psops_ctx *ctx, int *g, uint32_t *improved_words, float *pbest_loss);

/* The K losses currently held on the device, to dst (host or device). */
int psops_get_losses(psops_ctx *ctx, float *dst, int dst_on_device);

/*
 * Attach the quadratic stand-in fitness f(w) = sum_j dvec_j (w_j - tvec_j)^2
 * (device pointers, N floats each, borrowed; both NULL detaches).  Needs
 * PSOPS_QUADRATIC.  The summation order is fixed so that results are
 * reproducible bit for bit: fp32 terms dvec*(e*e) widened to fp64; four
 * consecutive terms added left to right; 32 such sums (128 elements) combined
 * by the butterfly a[l] += a[l ^ off], off = 16..1; tile sums added into 1024
 * slots (tile m -> slot m % 1024, increasing m, from +0.0); slots combined as
 * 32 butterflies of 32 and the 32 results added in order; rounded to fp32.
 */
int psops_set_quadratic(psops_ctx *ctx, const float *d_dvec, const float *d_tvec);

/* losses <- f(current weights) for every particle (the evaluation that
 * precedes the first sync). */
int psops_eval_quadratic(psops_ctx *ctx);

/*
 * (No counterpart in the paper: an addition for callers that cannot allocate.)
 * The quadratic fitness of K rows without any workspace and without a context:
 * d_loss[i] = f(row i of d_x), the same value, bit for bit, that
 * psops_eval_quadratic produces.  It is meant for code that has no way to get
 * device memory when it needs the value: inside a loop whose framework already
 * owns all of the GPU's memory through its caching allocator, in a plug-in that
 * is handed nothing but input and output buffers, or where cudaMalloc/cudaFree
 * are off limits because they stall every stream of the device.  The call
 * itself allocates nothing, on the host or on the device.
 *   d_x            K rows of stride ld (>= N) fp32, device pointer
 *   d_dvec, d_tvec N fp32 each, device pointers
 *   d_loss         K fp32, device pointer, written on the stream
 *   cuda_stream    a cudaStream_t (NULL = legacy default stream); work is only
 *                  enqueued
 * The intermediate tile sums go to an array of PSOPS_STATIC_SCRATCH_DOUBLES
 * doubles (8 MiB) that is built into the library and therefore occupies that
 * much memory on every GPU that loads it until the process exits.  A problem
 * with K * ceil(N/128) above that number is refused with PSOPS_ELIMIT and
 * nothing is launched.  The first call on each device looks the array's address
 * up (the device on which the pointers live must be current, then and in every
 * later call) -- make that first call outside any stream capture and at
 * start-up: if nothing else of this library has run on the device yet, it is
 * also the moment the CUDA runtime loads the library's device code and reserves
 * the 8 MiB, which may synchronise the device and, on a GPU with no memory
 * left, fail.  Such a failure is returned as PSOPS_ECUDA (there is no context
 * to hold a message; cudaGetLastError has been cleared).  All calls on a device share the array and it is not cleared
 * between calls (every slot that is read has been written by the same call);
 * calls that overlap in time on one GPU overwrite each other's partial results,
 * so keep them on one stream or order them yourself.
 * Errors: EINVAL (also: a buffer that is host memory, or device memory of a GPU
 * other than the current one), EALIGN (a pointer not 4-byte aligned), ELIMIT,
 * ECUDA.
 */
#define PSOPS_STATIC_SCRATCH_DOUBLES (1 << 20)
int psops_quadratic_fitness_static(const float *d_x, int64_t ld, int32_t K, int64_t N,
                                   const float *d_dvec, const float *d_tvec,
                                   float *d_loss, void *cuda_stream);

/* Checkpoint / resume of the small state: the sync counter (kept on the
 * device, so both calls wait for the stream) and pBest_loss (host pointers, one
 * float per particle of the whole swarm).  x, v, pbest are the caller's own
 * tensors; with PSOPS_GBEST_HISTORY also move the remembered row and loss
 * (psops_get_history / psops_set_history).  Restoring these into a new context
 * on the same tensors continues the run bit for bit: the random stream is a
 * function of (seed, sync counter, particle, element) only. */
int psops_get_state(psops_ctx *ctx, uint32_t *sync_step, float *pbest_loss);
int psops_set_state(psops_ctx *ctx, uint32_t sync_step, const float *pbest_loss);

/* Inertia weight of Eq. 5 as psops_sync would compute it (host only). */
float psops_inertia(const psops_config *cfg, int64_t t_iter);

/* Number of kernel launches this context has enqueued so far. */
int64_t psops_launch_count(const psops_ctx *ctx);

/* Static description of an error code. */
const char *psops_strerror(int code);

/* Text of the last CUDA error seen by this context ("" if none). */
const char *psops_last_error(const psops_ctx *ctx);

/* Waits for the stream, then frees the context (not the caller's buffers). */
int psops_destroy(psops_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* PSOPS_H */
