/*
 * gac.h -- C ABI of the B200 (sm_100a) library for the per-step hot path of
 * Gradient Alignment Control (GAC).
 *
 * Notation follows the paper: g is the aggregated gradient of the current
 * update step t (a list of per-parameter tensors, treated as one flattened
 * concatenation, App. A.1), d is the stored snapshot of the previous step's
 * gradient (App. A.2 "Memory footprint"), c_t their cosine (Eq. 1).
 *
 * Conventions for every entry point
 *   - returns a gac_status; never throws, aborts or traps; on failure
 *     gac_last_error() holds a message;
 *   - "device pointer" = address in the memory of the CUDA device the context
 *     was created for; "host pointer" = ordinary process memory;
 *   - g and d buffers belong to the CALLER; the library reads/writes them only
 *     inside gac_stats* / gac_project, on the stream given to that call;
 *   - the context owns its chunk table, per-CTA partial sums, decision record
 *     and a pinned host mirror of that record, and releases exactly those in
 *     gac_free();
 *   - one context serves one stream at a time and is not thread-safe.
 */
#ifndef GAC_H_
#define GAC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gac_ctx gac_ctx;   /* opaque, library-owned */

typedef enum {
    GAC_OK = 0,
    GAC_ERR_INVALID_ARG = 1,   /* null pointer, zero-length tensor, bad thresholds, ...      */
    GAC_ERR_DTYPE = 2,         /* unsupported (g, d) element-type pair                       */
    GAC_ERR_CUDA = 3,          /* a CUDA runtime call failed; message has the CUDA error     */
    GAC_ERR_STATE = 4,         /* calls out of order (project without stats, step going back)*/
    GAC_ERR_NONFINITE = 5,     /* NaN/Inf met in g or d; the step is reported as a violation  */
    GAC_ERR_TIMEOUT = 6        /* gac_decide_exchange: a peer's sums did not arrive within the limit
                                  (the only wait for another party in this library, bounded)    */
} gac_status;

typedef enum { GAC_F32 = 0, GAC_BF16 = 1 } gac_dtype;

/* The three regimes of Sec. 4.2 / Algorithm 1. */
typedef enum { GAC_REGIME_SAFE = 0, GAC_REGIME_PROJECT = 1, GAC_REGIME_VIOLATION = 2 } gac_regime;

typedef enum { GAC_MODE_ADAPTIVE = 0, GAC_MODE_FIXED = 1 } gac_mode;
typedef enum {
    GAC_STATE_RAW = 0,        /* d' = g, copied into the d buffers (the paper's rule)            */
    GAC_STATE_PROJECTED = 1,  /* d' = g' (variant)                                               */
    GAC_STATE_HOLD = 2,       /* d' = d  (variant)                                               */
    GAC_STATE_EXCHANGE = 3    /* d' = g as in RAW, but WITHOUT the copy: the two buffer sets swap
                                 roles after every step (see "Exchange mode" below)              */
} gac_state_mode;

/* Which of the two buffer sets of a context's list: the `g` pointers or the `d` pointers. */
typedef enum { GAC_SET_G = 0, GAC_SET_D = 1 } gac_buffer_set;

/* One parameter tensor: its gradient and its slot of the stored direction.
 * Both are device pointers to `numel` contiguous elements, caller-owned.
 * Any alignment is accepted; element-aligned is required, 16-byte aligned
 * bases take the vectorised path. */
typedef struct {
    void *g;
    void *d;
    uint64_t numel;
} gac_tensor;

/* Hyper-parameters.  Defaults of the paper: c_low 0.05, c_high 0.3 (App. C.3),
 * eps 1e-8 (App. A.1), beta 1 (App. A.2), adaptive mode, raw state, no clipping. */
typedef struct {
    double c_low, c_high;      /* Algorithm 1 inputs; ADAPTIVE mode needs 0 < c_low < c_high.
                                  c_high > 1 is legal and disables the skip branch.            */
    double eps;                /* added to sqrt(<g,g><d,d>) in the cosine (App. A.1); >= 0     */
    double beta;               /* gain of the orthogonal component (Eq. 3); finite             */
    int32_t mode;              /* gac_mode: ADAPTIVE = Eq. 5 with the three regimes;
                                  FIXED = Eq. 3 with (alpha_fixed, beta) on every step         */
    int32_t state_mode;        /* gac_state_mode: RAW d' = g (the paper's rule);
                                  PROJECTED d' = g'; HOLD d' = d; EXCHANGE d' = g by role swap  */
    double alpha_fixed;        /* gain of the parallel component in FIXED mode; 0 = remove it   */
    int32_t zero_on_violation; /* 0: leave g alone, the caller skips its optimizer step
                                  (Algorithm 1: theta_t = theta_{t-1}); 1: write g' = 0          */
    int32_t reserved;          /* must be 0 */
    double clip_max_norm;      /* > 0: global-norm clipping (Table 2 lists "Gradient clipping True")
                                  folded into the projection pass: what a safe or projection step
                                  sends on is scaled by min(1, clip_max_norm/(norm + clip_eps)),
                                  with the norm taken in closed form from the three sums, so the
                                  separate clipping pass of the optimizer is not needed.  0 = off.
                                  The stored direction is not clipped in state modes RAW, EXCHANGE
                                  and HOLD (it is the raw gradient, or left alone); PROJECTED stores
                                  d' = g' as written, hence clipped.                                */
    double clip_eps;           /* 1e-6 (the usual constant of global-norm clipping)                */
} gac_hparams;

/* What one step decided.  Lives on the device between gac_stats and
 * gac_project; copied to the host only when a host_out pointer is given. */
typedef struct {
    double dot, gg, dd;        /* <g,d>, <g,g>, <d,d> over the whole list (App. A.1)            */
    double cos;                /* c_t = dot / (sqrt(gg*dd) + eps); 0 when gg or dd is 0          */
    double alpha;              /* parallel gain used (Eq. 5: c_low/|c_t|); 1 when g is unchanged */
    double coef64;             /* (alpha - beta) * dot / dd : multiplier of d in the rank-one
                                  form g' = beta g + coef d (App. A.2)                          */
    float coef;                /* coef64 rounded once to binary32: the value the kernel uses    */
    int32_t regime;            /* gac_regime                                                    */
    int32_t nonfinite;         /* 1 if a sum was NaN/Inf: regime = VIOLATION, g and d untouched  */
    uint32_t staleness;        /* echoed metadata: the rule never reads it                      */
    uint64_t step;             /* Algorithm 1's t for which this record holds                    */
    double out_norm;           /* Euclidean norm of the gradient the step sends on, before clipping:
                                  sqrt(beta^2 gg + 2 beta coef dot + coef^2 dd) when projecting, sqrt(gg)
                                  when safe                                                       */
    double clip_scale;         /* factor applied by clipping (1 when off, not needed, or skipped) */
    uint64_t applied_steps;    /* optimizer updates applied so far by gac_project_adamw (skipped steps
                                  do not count); kept on the device across steps                  */
    uint32_t g_set;            /* gac_buffer_set that held this step's gradient (always GAC_SET_G
                                  outside exchange mode)                                          */
    uint32_t out_set;          /* gac_buffer_set that holds what the step sends on after
                                  gac_project: the same as g_set when g is updated in place or
                                  left alone; the other set when exchange mode wrote g' there     */
    uint32_t ref_lost;         /* exchange mode only: a non-finite step was closed, the stored
                                  direction is gone and the next step restarts from the zero
                                  reference (Algorithm 1's g_0 = 0)                               */
    uint32_t timed_out;        /* peer exchange only: a rank's numbers did not arrive within the limit;
                                  no decision was taken and the pass that follows writes nothing    */
} gac_result;

/* Fills *hp with the paper's defaults. */
void gac_default_hparams(gac_hparams *hp);

/*
 * gac_init -- build a context for one list of parameter tensors.
 * Presents the list as one logical flat vector (App. A.1: "flattened
 * concatenation of all trainable parameter gradients") WITHOUT copying: the
 * list is cut into fixed-size chunks, none spanning two tensors, and the chunk
 * table is uploaded once.  Re-create the context if the tensors move.
 *   out          host pointer, receives the context
 *   list         host pointer to n entries (device pointers inside), copied
 *   n            number of tensors, >= 1; every numel >= 1
 *   g_dtype/d_dtype  supported pairs: (F32,F32), (BF16,F32), and (BF16,BF16) -- a
 *                snapshot of half the size (App. A.2 "Memory footprint"), still an
 *                exact copy of the bfloat16 gradient.  state_mode EXCHANGE needs
 *                g_dtype == d_dtype (GAC_ERR_DTYPE otherwise)
 *   hp           host pointer; copied
 *   cuda_device  ordinal of the device that owns g and d
 * Allocates device and pinned memory (not capturable in a CUDA graph).
 * Errors: INVALID_ARG, DTYPE, CUDA.
 */
int gac_init(gac_ctx **out, const gac_tensor *list, uint32_t n, int g_dtype, int d_dtype,
             const gac_hparams *hp, int cuda_device);

/*
 * gac_stats -- one fused pass over g and d: the three inner products of
 * App. A.1, then the cosine with eps (App. A.1), the regime (Algorithm 1) and
 * the gains (Eq. 5, or Eq. 3 in FIXED mode), all left in a device-resident
 * decision record.  Sums are accumulated in binary64 in a fixed order: the
 * same inputs give bit-identical results run to run.
 *   step         Algorithm 1's t, counted from 1.  t = 1 means the stored
 *                direction is g_0 = 0: d is NOT read (it may be uninitialised)
 *                and the step is safe.  Must not go below the last step that
 *                gac_project completed.
 *   staleness    the lag tau of the behaviour policy; metadata only
 *   cuda_stream  a cudaStream_t (or NULL for the default stream)
 *   host_out     NULL: fully asynchronous, nothing leaves the device;
 *                else the stream is synchronised and the record copied there
 * Errors: INVALID_ARG, STATE, CUDA; NONFINITE only when host_out is given.
 */
int gac_stats(gac_ctx *ctx, uint64_t step, uint32_t staleness, void *cuda_stream,
              gac_result *host_out);

/*
 * Sharded form of gac_stats for data-parallel gradient sharding (App. A.1,
 * "Efficient computation under data parallelism"): each rank reduces its own
 * shard, ONE all-reduce sums three numbers, every rank takes the same decision.
 *   gac_stats_partial  writes this context's local (dot, gg, dd) to
 *                      sums_out, a DEVICE pointer to 3 doubles (8-byte aligned)
 *                      owned by the caller, and takes no decision;
 *   gac_decide         reads the GLOBAL (dot, gg, dd) from sums_in (device
 *                      pointer to 3 doubles, 8-byte aligned, e.g. after an
 *                      all-reduce on the same stream) and fills the decision record.
 * The collective between the two calls is the caller's.
 */
int gac_stats_partial(gac_ctx *ctx, uint64_t step, uint32_t staleness, void *cuda_stream,
                      double *sums_out);
int gac_decide(gac_ctx *ctx, void *cuda_stream, const double *sums_in, gac_result *host_out);

/*
 * Peer exchange: the sharded form WITHOUT a collective library.  App. A.1 needs
 * one all-reduce of three numbers per step and App. A.2 names it as GAC's one
 * extra synchronisation point.  Here the kernels do it themselves:
 *   gac_stats_exchange   reduces this rank's shard like gac_stats_partial; the
 *                        last CTA of that same kernel then stores the three sums
 *                        and the step number into this rank's slot of EVERY
 *                        rank's slot array (plain stores over NVLink for a peer,
 *                        no multicast, no bulk copy), and returns.  Nothing waits.
 *   gac_decide_exchange  one small kernel: waits until the slots of all ranks in
 *                        this rank's own array carry the step number, adds them
 *                        in RANK ORDER (every rank does the same additions in the
 *                        same order: bit-identical sums and decisions everywhere)
 *                        and fills the decision record, as gac_decide does.
 * Other work may be enqueued between the two calls.  The wait is bounded by the
 * timeout given to gac_exchange_attach (wall time on the device, plus a cap on
 * the number of polls); when it runs out the record is marked `timed_out`, no
 * decision is taken, and a following gac_project / gac_project_adamw writes
 * NOTHING (neither g nor d; in exchange state mode the stored direction is then
 * lost, as after a non-finite step).  With host_out the call returns
 * GAC_ERR_TIMEOUT and the step stays pending: gac_decide_exchange may be
 * repeated (the posted numbers stay where they are), or the step redone with
 * gac_stats_partial / gac_decide and the caller's own collective.
 *
 * gac_exchange_attach   rank, world (<= GAC_EXCHANGE_MAX_RANKS), and `slots`: a
 *                       host array of `world` DEVICE pointers, slots[r] = rank r's
 *                       slot array as addressable from this context's device
 *                       (slots[rank] is this rank's own).  Every array has
 *                       gac_exchange_bytes(world) bytes, is 32-byte aligned,
 *                       CALLER-owned, and must be zero-filled before the first
 *                       step and whenever step numbers start over.  How a peer's
 *                       array becomes addressable (peer access within a process,
 *                       an IPC or symmetric-memory mapping between processes) is
 *                       the caller's business.  timeout_ms = 0 means 1000.
 *                       Allocates a small table (not capturable).
 * Each array holds two sets of slots, used by odd and even steps in turn; that
 * is enough because a rank cannot post step t+2 before every peer has read the
 * slots of step t (it needs the peers' numbers of step t+1 first).
 * Errors: INVALID_ARG, STATE (not attached, calls out of order), CUDA, TIMEOUT.
 */
#define GAC_EXCHANGE_MAX_RANKS 1024
size_t gac_exchange_bytes(uint32_t world);
int gac_exchange_attach(gac_ctx *ctx, uint32_t rank, uint32_t world, void *const *slots, uint32_t timeout_ms);
int gac_stats_exchange(gac_ctx *ctx, uint64_t step, uint32_t staleness, void *cuda_stream);
int gac_decide_exchange(gac_ctx *ctx, void *cuda_stream, gac_result *host_out);

/*
 * gac_project -- one pass that reads g and d once and writes g' and d' in
 * place, steered by the decision record on the device (no host round trip):
 *   PROJECT regime   g'_i = beta g_i + coef d_i    (App. A.2 rank-one form;
 *                    one fused multiply-add per element when beta = 1, result
 *                    rounded to g's element type, nearest-even)
 *   SAFE             g untouched (Algorithm 1: ordinary update)
 *   VIOLATION        g untouched, or zeroed if zero_on_violation; the caller
 *                    skips its optimizer step (Algorithm 1: theta_t = theta_{t-1})
 *   every regime     d'_i = g_i, the raw gradient (state_mode RAW; EXCHANGE reaches the
 *                    same state without this copy, see "Exchange mode" below)
 *   nonfinite        neither g nor d is written (the same holds for a record
 *                    marked timed_out by gac_decide_exchange)
 * Must follow a gac_stats / gac_decide of the same step (else STATE).
 *   coef_override    host pointer to one float, or NULL.  When given, it
 *                    replaces the record's `coef` (used to compare outputs
 *                    "given the same coefficient").
 *   host_out         as in gac_stats
 */
int gac_project(gac_ctx *ctx, void *cuda_stream, const float *coef_override, gac_result *host_out);

/*
 * Exchange mode (state_mode GAC_STATE_EXCHANGE; g and d of the SAME element type).
 * App. A.2 keeps one snapshot of the previous gradient; refreshing it by a copy
 * costs a write of the whole vector on every step.  Here nothing is copied: the
 * buffers that held g simply BECOME the stored direction (they hold the raw
 * gradient already), and the buffers that held d become free.
 *   projection step   g' is written into the buffers that held d (read g, read d,
 *                     write once: 3 instead of 4 element transfers per parameter);
 *                     g itself is not modified
 *   safe / violation  nothing is read or written in the second pass; what a safe
 *                     step sends on is g, where it lies (read it, do not modify
 *                     it: it is the stored direction now).  zero_on_violation and
 *                     an active clip factor write their result (0, or s g) into
 *                     the buffers that held d.
 * After every gac_project / gac_project_adamw the roles swap: the NEXT gradient
 * must be written into the set that held d during this step.  The swap is
 * unconditional, so the caller can follow it without reading anything back:
 * step by step the gradient alternates between the two sets, starting with the
 * `g` pointers given to gac_init (gac_rebind starts over with the new `g`).
 * gac_next_gradient_set reports it (which set is g is a launch argument: a step
 * captured in a CUDA graph serves every second step).  The record says where the outgoing gradient
 * is (`out_set`).  A non-finite step writes nothing; since the roles swap all the
 * same, the stored direction is lost with it and the following step is taken
 * against the zero reference (`ref_lost`), as the first step is.
 */
int gac_next_gradient_set(const gac_ctx *ctx, int *set_out /* host pointer: gac_buffer_set */);

/*
 * The step after the path: the update handed straight to the optimizer.
 * Algorithm 1 ends each safe or projection step with theta_t = theta_{t-1} +
 * eta g' and the paper trains with AdamW (Table 2: lr 1e-6, betas (0.9, 0.999),
 * eps 1e-8, weight decay 1e-2, gradient clipping on).  gac_project_adamw is
 * gac_project and that optimizer step in ONE pass: it reads g, d, p, m, v once,
 * writes d' = g and the new p, m, v, and never writes g' back (g is left as it
 * was), which saves the separate optimizer pass over g'.
 *     g' = clip_scale (beta g + coef d)   (projection)   or  clip_scale g   (safe)
 *     p <- p (1 - lr wd);  m <- b1 m + (1-b1) g';  v <- b2 v + (1-b2) g'^2
 *     p <- p - lr/(1-b1^t) * m / (sqrt(v)/sqrt(1-b2^t) + eps),  t = applied_steps + 1
 * A violation step changes neither p, m nor v (Algorithm 1: theta_t = theta_{t-1})
 * and does not advance t; a non-finite step changes nothing at all.
 *
 * gac_attach_adamw   binds the optimizer state of every tensor of the context's
 *                    list (same order, same numel; float32 device buffers, CALLER-
 *                    owned) and sets the number of updates applied so far
 *                    (0 for a fresh optimizer).  Allocates a second table.
 * gac_project_adamw  replaces gac_project for this step (same call order rules).
 *                    Needs state_mode RAW or EXCHANGE (then d' is not written either:
 *                    the roles swap).  opt is a host pointer, copied.
 * Errors: INVALID_ARG, STATE (not attached, no decision pending), CUDA.
 */
typedef struct {
    void *p;   /* parameter            */
    void *m;   /* first moment         */
    void *v;   /* second moment        */
} gac_opt_tensor;
typedef struct {
    double lr, beta1, beta2, eps, weight_decay;
} gac_adamw;
void gac_default_adamw(gac_adamw *opt);   /* Table 2 values */
int gac_attach_adamw(gac_ctx *ctx, const gac_opt_tensor *list, uint32_t n, uint64_t applied_steps);
int gac_project_adamw(gac_ctx *ctx, void *cuda_stream, const gac_adamw *opt,
                      const float *coef_override, gac_result *host_out);

/* Releases what the context owns (never g or d).  NULL is accepted. */
int gac_free(gac_ctx *ctx);

/* Message of the last failure on this context; with ctx == NULL, of the last
 * failed gac_init on the calling thread.  Never NULL. */
const char *gac_last_error(const gac_ctx *ctx);

/*
 * Launch geometry (no counterpart in the paper; tuning only).  Values <= 0
 * keep the default.  Must be called before the first gac_stats.
 *   chunk_elems     elements per chunk (multiple of 1024)
 *   ctas_per_sm     resident CTAs per SM the grid is sized for
 * Changing them changes the summation order, hence the last bits of the sums.
 */
int gac_set_launch(gac_ctx *ctx, int chunk_elems, int ctas_per_sm);

/*
 * gac_rebind -- point an existing context at moved buffers (a framework that
 * re-allocates its gradient tensors changes their addresses, not their sizes).
 * Same number of tensors and the same numel each; the step counter, the
 * hyper-parameters and the device-resident record are kept, so the state in
 * the new d buffers is taken as the stored direction of the next step.  Only
 * between steps (not between gac_stats and gac_project).  Frees and
 * re-allocates the chunk table, which synchronises the device.
 * Errors: INVALID_ARG, STATE, CUDA.
 */
int gac_rebind(gac_ctx *ctx, const gac_tensor *list, uint32_t n);

/* Facts about the context: total elements, chunks, grid size, kernel launches so far. */
typedef struct {
    uint64_t total_elems;
    uint64_t n_chunks;
    uint32_t n_tensors;
    uint32_t grid;
    uint32_t threads;
    uint32_t chunk_elems;
    uint64_t launches;
    uint32_t misaligned_tensors;
    uint32_t reserved;
} gac_info;
int gac_get_info(const gac_ctx *ctx, gac_info *out);

/*
 * gac_stats_static -- gac_stats for callers that must not allocate.
 * (No counterpart in the paper: it computes exactly what gac_stats computes;
 * only where the work memory comes from differs.)
 *
 * Who needs it: code that runs where asking the driver for device memory is
 * off limits -- inside a region whose memory is wholly owned by a framework's
 * pool (so a cudaMalloc could fail or fragment it), on a latency-critical path
 * where the implicit device-wide synchronisation of cudaMalloc/cudaFree is
 * unacceptable, or in a process that was told to keep a fixed memory footprint.
 * gac_init allocates a chunk table, partial sums and a pinned mirror; this
 * entry point needs no context, calls no allocating CUDA routine and does not
 * use the host heap either (the host image of the table sits in a fixed 2 MiB
 * buffer of the library, filled under a lock).
 *
 * How: the chunk table, the per-CTA partial sums and the arrival ticket live
 * in an array that is part of the library image: GAC_STATIC_SCRATCH_BYTES
 * (about 2.1 MiB) on EVERY device that loads the library, held until the
 * process exits.  The list is cut into chunks of 16384 elements, none spanning
 * two tensors; at most GAC_STATIC_MAX_CHUNKS chunks fit (65536: up to about
 * 1.07e9 elements; every tensor costs at least one chunk).  A list that needs
 * more is refused with GAC_ERR_INVALID_ARG and a message; use gac_init then.
 *
 *   list, n, g_dtype, d_dtype, hp, step, staleness   as in gac_init / gac_stats
 *                    (list is a host pointer; g and d inside are device
 *                    pointers, caller-owned, only read)
 *   cuda_device      device that owns g, d and result_dev (0..63)
 *   cuda_stream      stream for the two small copies and the one kernel launch
 *   result_dev       DEVICE pointer, caller-owned, 8-byte aligned: receives the
 *                    gac_result of this step when the stream reaches that point
 *                    (every field is written; applied_steps and ref_lost read 0).
 *                    Nothing is copied back to the host.
 *
 * Host-side behaviour: the chunk table is copied to the device from ordinary
 * (pageable) library memory.  Such a copy makes the calling thread wait until
 * the work queued earlier on cuda_stream has drained and the table has been
 * staged; the reduction itself then runs asynchronously.  A caller that cannot
 * afford that wait gives the call a stream of its own and orders it with events.
 *
 * The first call on each device looks up the device address of the built-in
 * array (once, with that device current).  No call may be made on a stream that
 * is being captured into a CUDA graph: a replay would copy the table from the
 * library's host buffer as it stands THEN, after other calls have rewritten it.
 * Such a call is refused with GAC_ERR_STATE and nothing is enqueued.
 *
 * All calls on a device share the one array, and it keeps what the previous
 * call left: each call re-zeroes the ticket and rewrites the table on its
 * stream before launching.  Two calls whose GPU work overlaps (different
 * streams without ordering, or two host threads) race on that array and give
 * wrong sums: order them on one stream or with events.
 * Only the statistics pass has this form; gac_project still wants a context.
 * Errors: INVALID_ARG, DTYPE, STATE (stream is capturing), CUDA (message via
 * gac_last_error(NULL)).
 */
#define GAC_STATIC_MAX_CHUNKS 65536
#define GAC_STATIC_SCRATCH_BYTES (256 + 62976 + GAC_STATIC_MAX_CHUNKS * 32)
int gac_stats_static(const gac_tensor *list, uint32_t n, int g_dtype, int d_dtype,
                     const gac_hparams *hp, uint64_t step, uint32_t staleness, int cuda_device,
                     void *cuda_stream, gac_result *result_dev);

#ifdef __cplusplus
}
#endif
#endif /* GAC_H_ */
