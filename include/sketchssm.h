/*
 * sketchssm.h -- C ABI of the SketchSSM decode hot path for NVIDIA B200 (sm_100a).
 *
 * SketchSSM keeps the full recurrent state S (K x V, fp32) of a linear-attention
 * layer exact, but lets the decode steps between two state updates read only a
 * compact sketch U = S^T Omega (V x r) of it.  One window of L tokens is
 * (Algorithm 1, inference part):
 *     L-1 times  sketchssm_decode_step   : append token, o = U C q~ + o_buffer
 *     once       sketchssm_state_update  : append token, replay the L buffered
 *                                          tokens into S, o = S^T q, U = S^T Omega
 * sketchssm_full_read_decode is the exact decode that reads all of S every step
 * (the buffered-replay baseline of Eq. 4); it is kept as the in-library baseline.
 *
 * Recurrences (Section 3.1, Eq. 1-4), per (batch b, head h):
 *   S_t = M_t S_{t-1} + beta_t k_t v_t^T,  M_t = (I - beta_t k_t k_t^T) D_t  (GDN, KDA)
 *                                          M_t = D_t                         (Mamba-2)
 *   D_t = a_t I (Mamba-2), alpha_t I (GDN), Diag(g_t) (KDA)
 *   o_t = S_0^T q~_t + sum_{s<=t} a_s v_s,  q~_t = M_{1:t}^T q_t,
 *   a_s = beta_s <M_{s+1:t} k_s, q_t>.
 *
 * General rules
 *   - Every pointer in sketchssm_buffers and every tensor argument of the three
 *     hot-path calls is a DEVICE pointer on the configured device, owned by the
 *     caller, 16-byte aligned, densely packed in the layouts below.  The library
 *     allocates no device memory and keeps no copy of any tensor.
 *   - The hot-path calls only enqueue work on `stream` (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and return; they never synchronise.
 *   - Return value: SKETCHSSM_OK (0) or a negative sketchssm_status.  Nothing
 *     throws, aborts or traps.  Kernels bound every wait; a wait that runs out
 *     records a code in the caller's status word (see sketchssm_buffers.status).
 *   - The window phase is the caller's: `n_before` (tokens already buffered) is
 *     the same for the whole batch.
 *   - Every call that touches the GPU makes config.device the calling thread's current CUDA device
 *     and leaves it current on return; a caller that drives several GPUs from one thread must not
 *     assume that its previous device is still selected.
 *
 * Layouts (B = batch, H = heads, K = dk, V = dv, r = rank, L = buf_len; "io" is
 * float or bfloat16 as configured):
 *   state  S      [B][H][K][V]  fp32
 *   sketch U      [B][H][r][V]  fp32   (U^T of the paper's V x r matrix: row g is S^T omega_g); bfloat16 with
 *                                      config.sketch_dtype = SKETCHSSM_BF16 (then C is bfloat16 too)
 *   omega  Omega  [H][K][r]     fp32   (fixed offline, shared by the batch)
 *   coef   C      [H][r][K]     fp32   (fixed offline coefficient map, Eq. 10), or with config.coef_per_seq
 *                 [B][H][r][K]  fp32   (state-dependent map, written by sketchssm_state_update)
 *   ring          [B][H] blocks of sketchssm_sizes.ring_head_bytes, each
 *                   k     [L][K] io
 *                   v     [L][V] io
 *                   beta  [L]    fp32
 *                   decay [L]    fp32 (Mamba-2 a_t, GDN alpha_t)  or  [L][K] io (KDA g_t)
 *   token inputs  q,k [B][H][K] io;  v [B][H][V] io;  beta [B][H] fp32;
 *                 decay [B][H] fp32 (Mamba-2, GDN) or [B][H][K] io (KDA)
 *   output        o [B][H][V] fp32 or bfloat16 (config.out_dtype)
 */
#ifndef SKETCHSSM_H_
#define SKETCHSSM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum sketchssm_kind { SKETCHSSM_MAMBA2 = 0, SKETCHSSM_GDN = 1, SKETCHSSM_KDA = 2 };
enum sketchssm_dtype { SKETCHSSM_F32 = 0, SKETCHSSM_BF16 = 1 };

typedef enum sketchssm_status {
    SKETCHSSM_OK = 0,
    SKETCHSSM_INVALID_ARG = -1,       /* null pointer, misaligned pointer, n out of range, bad flag mix */
    SKETCHSSM_UNSUPPORTED_SHAPE = -2, /* shape outside the compiled set (see sketchssm_create) */
    SKETCHSSM_NOT_BOUND = -3,         /* hot-path call before sketchssm_bind */
    SKETCHSSM_CUDA_ERROR = -4,        /* a CUDA runtime call failed (launch, attribute, device) */
    SKETCHSSM_DEVICE_TIMEOUT = -5     /* read back from the status word: a bounded device wait ran out */
} sketchssm_status;

/* flags of sketchssm_state_update */
#define SKETCHSSM_NO_SKETCH 0x1u      /* do not write U (the flush kernel without the sketch) */
/* flags of sketchssm_decode_step / sketchssm_full_read_decode */
#define SKETCHSSM_NO_APPEND 0x1u      /* use the token for this step's output but do not store it in the ring */

typedef struct sketchssm_config {
    int32_t kind;       /* sketchssm_kind */
    int32_t batch;      /* B >= 1 */
    int32_t heads;      /* H >= 1 */
    int32_t dk;         /* K: 64 or 128 */
    int32_t dv;         /* V: 64, 80 (with dk = 128) or 128 */
    int32_t rank;       /* r: 1..64 */
    int32_t buf_len;    /* L: 4..64, multiple of 4 */
    int32_t io_dtype;   /* sketchssm_dtype of q, k, v, KDA g and of the ring's k, v, g */
    int32_t out_dtype;  /* sketchssm_dtype of o */
    int32_t device;     /* CUDA device ordinal */
    int32_t coef_per_seq;   /* 0: C is the fixed offline map [H][r][K], an input shared by the batch (Eq. 10).
                               1: C is the state-dependent map (Eq. 9 with the ridge of Appendix A.2.2), one per
                                  (batch, head), [B][H][r][K]; every sketchssm_state_update that writes the sketch
                                  rebuilds it from the updated state, and the decode step reads it beside U.
                                  Omega must then have orthonormal columns (the appendix's assumption). */
    int32_t coef_pivots;    /* coef_per_seq = 1: pivot count P of the low-rank-plus-diagonal state metric
                               (Eq. 30-37; the paper uses 4; 1..8), or 0 for the exact ridge solve (Eq. 29) */
    float ridge_lambda;     /* coef_per_seq = 1: ridge lambda > 0 (the paper uses 0.1) */
    int32_t sketch_dtype;   /* sketchssm_dtype of the stored sketch U and coefficient map C: SKETCHSSM_F32 (default) or
                               SKETCHSSM_BF16, the storage the paper's traffic model assumes (T_G = 2 G (V + K) bytes per
                               non-flush read, Appendix D).  U is rounded to bfloat16 once, when the flush stores it; all
                               arithmetic stays fp32.  The fixed offline map (coef_per_seq = 0) is then handed over as
                               bfloat16 [H][r][K]; the state-dependent map (coef_per_seq = 1) is built from the sketch as
                               stored (the rounded rows) and rounded to bfloat16 once, when it is stored [B][H][r][K].
                               Only the default one-kernel decode is available with bfloat16 storage. */
    int32_t erase_factors;  /* GDN / KDA only.  0 (default): the decode step forms the effective query q~_t by the backward
                               sweep over the ring and then c_t = C q~_t.  1: it forms c_t from projected erase vectors
                               (Appendix C.2, Eq. 44-45): every appended token leaves f_s = beta_s [C (d_[s] * k_s) -
                               sum_{j<s} f_j <l_j(s), k_s>] in R^r in the `erase` buffer, and c_t = C (d_[t] * q_t) -
                               sum_{s<=t} f_s <l_s(t), q_t> with <l_s(t), y> taken from the stored ring keys and the
                               cumulative decays (Eq. 46).  Exact for the map in force during the window (the same c_t up
                               to rounding order); costs r stored elements (fp32 or bfloat16, like the sketch) per buffered token and step.
                               Needs rank % 4 == 0 (% 8 with bfloat16 storage) and
                               buf_len <= 32; only the default one-kernel decode supports it. */
} sketchssm_config;

typedef struct sketchssm_sizes {
    size_t state_bytes, sketch_bytes, ring_bytes, omega_bytes, coef_bytes;
    size_t status_bytes;     /* size of the status block: 4 status ints, then the update kernel's tile-scheduler
                                counters (4 + heads ints), rounded up to 16 bytes */
    size_t work_bytes;       /* per-head weight hand-off between the two decode kernels: B*H*(K+L) floats */
    size_t ring_head_bytes;  /* stride of one (b, h) ring block */
    size_t ring_v_offset, ring_beta_offset, ring_decay_offset; /* byte offsets inside a ring block (k is at 0) */
    size_t alignment;        /* required alignment of every pointer (16) */
    size_t erase_bytes;      /* erase_factors = 1: B*H*L*rank elements of the sketch's storage type (else 0) */
} sketchssm_sizes;

typedef struct sketchssm_buffers {
    void* state;   /* S      */
    void* sketch;  /* U      */
    void* ring;    /* ring   */
    void* omega;   /* Omega  */
    void* coef;    /* C      */
    void* status;  /* status_bytes, zero-initialised by the caller.  int32[0..3]: [0] first device fault code
                      (0 = none), [1] which wait, [2..3] reserved; kernels only ever write non-zero codes
                      there and sketchssm_read_status reads them back.  The ints after them are counters
                      of the state-update kernel's tile scheduler: every launch leaves them zero again,
                      and the caller never touches them after the initial zeroing.  Two state updates that
                      overlap on the GPU therefore need separate contexts with separate status blocks
                      (as they do anyway: they would update the same state). */
    void* work;    /* work_bytes of scratch for the decode calls (contents are transient: written and
                      consumed inside one call; calls that overlap on the GPU need separate contexts
                      with separate work buffers) */
    void* head_rank; /* optional (may be NULL): int32[H], the sketch rank of every head index of this layer, as an
                      offline rank allocation assigns it (Appendix E): 1..rank = the head uses that many columns
                      of Omega (its sketch rows and coefficient rows beyond them are ignored and its decode step
                      fetches only that many); 0 = a dense-fallback head whose decode step reads the full state
                      exactly, inside the same launch.  Layouts keep the configured `rank` as their row stride.
                      Only the default one-kernel decode supports the table. */
    void* erase;   /* erase_factors = 1: erase_bytes, [B][H][L][rank] in the sketch's storage type (fp32, or bfloat16: then
                      every vector is rounded once, where it is stored, and rank % 8 = 0): slot s of a (b, h) block holds f_s of the token
                      in ring slot s (written by the decode step that appends the token, read by the later steps of the
                      window; a state update empties the ring and with it these slots).  Contents need no
                      initialisation.  Ignored (may be NULL) when erase_factors = 0. */
} sketchssm_buffers;

typedef struct sketchssm_ctx sketchssm_ctx; /* host-only metadata; owns no device memory */

/* Validate the configuration and create a context.  Host-only (no CUDA call).
 * Supported: dk in {64,128}, dv in {64,128}, 1 <= rank <= 64, buf_len in 4..64 and a
 * multiple of 4, any kind / dtype combination.  Returns INVALID_ARG / UNSUPPORTED_SHAPE. */
int sketchssm_create(const sketchssm_config* cfg, sketchssm_ctx** out);
int sketchssm_destroy(sketchssm_ctx* ctx);

/* Byte sizes and ring sub-offsets for this configuration.  Host-only. */
int sketchssm_query_sizes(const sketchssm_ctx* ctx, sketchssm_sizes* out);

/* Record the caller's device buffers (the first seven required, 16-byte aligned; head_rank optional, 4-byte aligned).  The context
 * stores the pointers only; the caller keeps ownership and must keep them alive.
 * Between calls on a context its sketch is written by sketchssm_state_update only.  The library's kernels
 * are launched with programmatic dependent launch, and a decode step that does not directly follow a state
 * update (or a bind) of its own context requests sketch rows before it waits for its predecessor in the
 * stream.  So a sketch buffer must not be shared between contexts, and work of the caller that writes the
 * sketch (a kernel, a copy that restores a checkpoint) must be followed by sketchssm_bind, which makes
 * the next decode step wait first, or by a stream synchronisation.  A decode step recorded into a stream
 * capture always waits first (a replayed graph may follow a state update that is still running).  With the
 * tune key "pdl" = 0 every kernel waits for its predecessor as usual. */
int sketchssm_bind(sketchssm_ctx* ctx, const sketchssm_buffers* bufs);

/* Flush step of Algorithm 1: (optionally) append the current token, replay every buffered
 * token into S exactly (Eq. 3), then o = S^T q from the updated state and U = S^T Omega
 * (Eq. 7) while the updated tile is still on chip, so S is read once and written once.
 *   n_before : tokens already in the ring, 0..L (0..L-1 when a token is given).
 *   k, v, beta, decay : the current token, all given or all NULL.  When given it is
 *              replayed last (it need not be stored: the ring is empty afterwards).
 *   q, out   : both given or both NULL; out = S_new^T q (exact output of the flush step).
 *   flags    : SKETCHSSM_NO_SKETCH leaves U untouched.
 * With n_before = 0 and no token, S is left untouched and only U (and out) are produced:
 * this builds the initial sketch from a prefilled state.
 * With config.coef_per_seq = 1 every call that writes U also rebuilds the coefficient maps C of all (batch, head)
 * pairs from S_new and U (a second kernel of the same call: the map needs the complete sketch before it can be
 * contracted with the state, so S_new is read once more): mu = ||S_new||_F^2 / K, then either the exact ridge form
 * C = (U^T U + lambda mu I)^{-1} U^T S_new^T or, with P = config.coef_pivots > 0, the approximation of Appendix A.2.2
 * (Gram-Schmidt basis Q of the first min(r, P) sketch columns, L = S Q / sqrt(mu), residual diagonal d, Woodbury
 * solve of the P x P system).
 * After the call the caller's ring count is 0. */
int sketchssm_state_update(sketchssm_ctx* ctx, int n_before, const void* q, const void* k,
                           const void* v, const void* beta, const void* decay, void* out,
                           uint32_t flags, void* stream);

/* Non-flush decode step of Algorithm 1: store the token in ring slot n_before, form q~_t and
 * the buffer weights from the n_before+1 buffered tokens (Eq. 4), c_t = C q~_t, and write
 * o = U c_t + sum_s a_s v_s.  S is not touched.  n_before in 0..L-1; all pointers required.
 * After the call the caller's ring count is n_before + 1 (unless SKETCHSSM_NO_APPEND).
 * With config.coef_per_seq = 1 the head's own map C[b][h] is read (r * K * 4 more bytes per head and step); only the
 * default one-kernel decode supports this ("decode_impl" = 0 and sketchssm_decode_step_static return
 * SKETCHSSM_UNSUPPORTED_SHAPE). */
int sketchssm_decode_step(sketchssm_ctx* ctx, int n_before, const void* q, const void* k,
                          const void* v, const void* beta, const void* decay, void* out,
                          uint32_t flags, void* stream);

/* One step of Algorithm 1 for a batch whose sequences are at different window phases (continuous batching: sequences
 * join and flush at different times).  `phase` is a DEVICE array int32[B], one entry per batch entry b:
 *     phase[b] = n >= 0       the sequence takes a non-flush decode step with n tokens already buffered (0..L-1):
 *                             exactly sketchssm_decode_step for its heads;
 *     phase[b] = -(n + 1) < 0 the sequence takes the flush step with n tokens buffered (0..L-1) plus the current one:
 *                             exactly sketchssm_state_update with the token, q and out for its heads (the flush may
 *                             come before the ring is full).
 * The call enqueues the decode kernel (which skips the flushing sequences) and the flush kernel (which skips the
 * others; with per-sequence phases the CUDA-core flush kernel is used), then, with config.coef_per_seq, the
 * coefficient-map kernel for the flushed sequences.  All token pointers are required; `out` receives every
 * sequence's output.  The caller keeps the counts: after the call a sequence with phase n >= 0 holds n + 1 tokens,
 * a flushed one none.  `phase` is read by the kernels, so it must not change until they have run. */
int sketchssm_step_mixed(sketchssm_ctx* ctx, const int32_t* phase, const void* q, const void* k, const void* v,
                         const void* beta, const void* decay, void* out, uint32_t flags, void* stream);

/* Exact decode step that reads the whole state: o = S_0^T q~_t + sum_s a_s v_s (Eq. 4).
 * Same arguments and ring behaviour as sketchssm_decode_step; U and C are not read.
 * By default both decode calls run as one kernel with a warp per (batch, head) and leave `work` alone; with the
 * tune key "decode_impl" = 0 they run as two kernels, the first of which forms the buffer weights a_s and the
 * coefficients (c_t, or q~_t for the full read) into `work` and the second the weighted sum of rows. */
int sketchssm_full_read_decode(sketchssm_ctx* ctx, int n_before, const void* q, const void* k,
                               const void* v, const void* beta, const void* decay, void* out,
                               uint32_t flags, void* stream);

/* Size of the library-owned device array used by sketchssm_decode_step_static. */
#define SKETCHSSM_STATIC_WORK_BYTES (4u << 20)

/* (The paper has no counterpart of this entry point: it exists for deployment, not for the method.)
 * sketchssm_decode_step for callers that cannot provide scratch memory and must not trigger an allocation:
 * an engine whose device memory pool is carved up once at start-up, a plug-in that only ever receives its
 * tensors, code inside a region where an allocation would synchronise the device.  Same arguments, same
 * result (up to floating-point summation order) and same ring behaviour as sketchssm_decode_step, always as
 * the two-kernel decode; the per-head weight hand-off between the two kernels lives in a device array that
 * belongs to the library (SKETCHSSM_STATIC_WORK_BYTES = 4 MiB, held by every GPU that loads the library until
 * the process exits) instead of in sketchssm_buffers.work, which this call never touches.  The call itself
 * allocates nothing, on the host or on the device.
 *   - Limit: batch * heads * (dk + buf_len) * 4 bytes must fit in the array, otherwise the call returns
 *     SKETCHSSM_UNSUPPORTED_SHAPE and launches nothing.
 *   - The first call made on a device looks up the array's address on that device (one runtime query, no
 *     allocation); make that first call outside any stream capture.
 *   - All contexts, streams and threads share the one array.  It keeps whatever the last call left in it; the
 *     kernels overwrite every element they read, so nothing has to be cleared.  Two calls that overlap on the
 *     GPU (different streams, or different contexts on the same device) race on it: serialise them. */
int sketchssm_decode_step_static(sketchssm_ctx* ctx, int n_before, const void* q, const void* k,
                                 const void* v, const void* beta, const void* decay, void* out,
                                 uint32_t flags, void* stream);

/* Device staging for one step's token tensors, caller-owned, same shapes/dtypes as the token
 * arguments of the hot-path calls (q,k [B][H][K] io; v [B][H][V] io; beta [B][H] fp32; decay;
 * out [B][H][V]).  Used only by sketchssm_step_host. */
typedef struct sketchssm_staging {
    void *q, *k, *v, *beta, *decay, *out;
} sketchssm_staging;

enum sketchssm_op { SKETCHSSM_OP_DECODE = 0, SKETCHSSM_OP_FULL_READ = 1, SKETCHSSM_OP_UPDATE = 2 };

/* One step of Algorithm 1 with HOST token tensors: enqueue on `stream` the host->device copies of
 * q, k, v, beta, decay into `staging`, the chosen hot-path call (decode step, full-read decode, or
 * state update with the token and the exact output), and the device->host copy of the output into
 * `host_out`.  Host buffers should be page-locked for the copies to be asynchronous; they must stay
 * valid until the stream has passed this step.  Same n_before / flags rules as the underlying call. */
int sketchssm_step_host(sketchssm_ctx* ctx, int op, int n_before, const void* host_q, const void* host_k,
                        const void* host_v, const void* host_beta, const void* host_decay, void* host_out,
                        const sketchssm_staging* staging, uint32_t flags, void* stream);

/* Copy the status word back (synchronises `stream`).  Returns SKETCHSSM_OK if no kernel
 * recorded a fault, SKETCHSSM_DEVICE_TIMEOUT otherwise; `detail`, if not NULL, receives the
 * four status ints. */
int sketchssm_read_status(sketchssm_ctx* ctx, int32_t detail[4], void* stream);

/* Self-test of the failure-reporting path (no counterpart in the paper).  Every device wait of the hot-path kernels
 * is bounded and reports through the status block when its limit is reached; in normal operation none ever does.
 * This call launches one warp that waits, for at most `poll_limit` polls (1..65536), on a barrier phase that nothing
 * completes -- no copy is issued, so nothing is in flight when it gives up -- and then records the fault code 4 with
 * `where` as the place.  Afterwards sketchssm_read_status returns SKETCHSSM_DEVICE_TIMEOUT with detail = {4, where, ..}.
 * The status block keeps its first fault: zero its first four ints before going on with normal calls.  The GPU
 * context stays usable; nothing traps or hangs. */
int sketchssm_selftest_wait_timeout(sketchssm_ctx* ctx, int poll_limit, int where, void* stream);

/* Text of the CUDA runtime error behind the most recent SKETCHSSM_CUDA_ERROR of this context. */
const char* sketchssm_last_cuda_error(const sketchssm_ctx* ctx);

/* Number of kernels the last hot-path call on this context launched (host counter). */
int sketchssm_last_launch_count(const sketchssm_ctx* ctx);

/* Optional launch tuning, host-only.  Keys: "decode_batches_per_cta" (batch entries one CTA of
 * the two-kernel decode serves for its head; 0 = library default), "decode_stages" (1 or 2 shared-memory
 * stages per lane group of the two-kernel decode; for the warp-specialised update kernels an upper
 * bound >= 2 on their shared-memory stages of state rows; 0 = library default), "decode_warps_per_cta",
 * "decode_max_warps_per_sm" (also caps the update kernels' CTAs per SM), "update_impl" (0 = warp-specialised
 * tensor-core kernels where their shape limits allow and CUDA cores otherwise, the default; 1 = CUDA cores
 * only; 3 = as 0 but the single-group tensor-core kernel for Mamba-2 and CUDA cores for the delta-rule kinds),
 * "decode_impl" (0 = two kernels; 1 = one fused kernel with a warp per head, the default), "pdl"
 * (1 = programmatic dependent launch, the default).
 * Results depend on these only through floating-point summation order. */
int sketchssm_tune(sketchssm_ctx* ctx, const char* key, int value);

const char* sketchssm_status_string(int status);
const char* sketchssm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SKETCHSSM_H_ */
