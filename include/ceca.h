/*
 * ceca.h -- C ABI of the DSGD-CECA hot path for one NVIDIA B200 (sm_100a).
 *
 * n simulated agents are the rows of dense row-major fp32 matrices X (the models x_i),
 * Y (the auxiliary models y_i) and G (the stochastic gradients e_i), each n x d with a
 * leading dimension ld >= d counted in elements (for full bandwidth make ld a multiple of 32, so
 * that every row starts on a 128-byte line: with rows of 25.6M floats this is worth ~4 %).  One call applies one iteration of
 * DSGD-CECA (Algorithm 1), or several CECA consensus rounds (Algorithm 2), to all agents.
 *
 * Conventions shared by every entry point
 *   - Agent indices are 0-based: the paper's agent p is row p-1, so a "paper-odd" agent
 *     is an even row.
 *   - Pointers named X, Y, G, A, labels, *_out and workspace are DEVICE pointers unless the
 *     function name ends in _host.  The caller owns every buffer; the library allocates no
 *     device memory and never frees anything.  What it keeps between calls is small and holds no
 *     problem data: per-device constants (SM count, kernel attributes set once) and a cache of
 *     encoded TMA tensor maps keyed on (pointer, n, d, ld).  Two entry points go further and say
 *     so below: dsgd_logreg_grad_static (a fixed scratch buffer inside the library) and
 *     ceca_gossip_sgd_step_host (internal streams, created and destroyed per call).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Device entry points only enqueue work: they do not synchronise and return as soon
 *     as the launches are queued.
 *   - Argument errors are reported synchronously, before anything is launched, through the
 *     return value.  Nothing aborts or traps; no exception crosses this boundary.
 *   - `variant` is CECA_1P (pairwise exchange, even n only) or CECA_2P (send to one agent,
 *     receive from another; any n >= 1).
 *   - `k` is the iteration counter of Algorithm 1; the round is r = k mod tau with
 *     tau = ceil(log2 n).  k may be any value in [0, 2^63).
 */
#ifndef CECA_H_
#define CECA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { CECA_1P = 1, CECA_2P = 2 } ceca_variant_t;

typedef enum {
  CECA_OK = 0,
  CECA_ERR_INVALID_ARG = 1, /* NULL where data is needed, n < 1, d < 1, ld < d, k < 0, ...       */
  CECA_ERR_ODD_N_1P = 2,    /* CECA-1P is defined for even n only (Sec. 3.2)                     */
  CECA_ERR_ALIGNMENT = 3,   /* the fused consensus kernel needs 16-byte aligned rows             */
  CECA_ERR_UNSUPPORTED = 4, /* e.g. crossed aliasing of X/Y buffers, a fused kernel outside its range of n */
  CECA_ERR_WORKSPACE = 5,   /* workspace NULL or smaller than ceca_workspace_bytes says          */
  CECA_ERR_CUDA = 6,        /* a CUDA runtime / driver call failed (launch, copy, map encode)    */
  CECA_ERR_STATIC_SCRATCH = 7 /* dsgd_logreg_grad_static: the problem needs more scratch than the
                                 built-in buffer holds; use dsgd_logreg_grad with a workspace       */
} ceca_status_t;

/*
 * Everything Algorithm 1 derives from (n, k) for one iteration.
 * Sec. 3.1 "Auxiliary variables": n-1 = (delta_0 ... delta_{tau-1})_2 with delta_0 the most
 * significant digit; n_0 = 0, n_{r+1} = 2 n_r + delta_r.
 * Algorithm 1: delta_r = 1 -> the message is built from x, a = 1/2, b = n_r/(2 n_r + 1);
 *              delta_r = 0 -> the message is built from y, a = (n_r+1)/(2 n_r+1), b = 1/2.
 * n = 1 (not covered by the paper): tau = 0, r = 0, a = b = 1, nobody to talk to.
 */
typedef struct {
  int32_t n, tau, r, delta, n_r;
  int32_t payload;                    /* 0: z = x (delta = 1);  1: z = y (delta = 0)          */
  int32_t a_num, a_den, b_num, b_den; /* exact weights (not necessarily in lowest terms)      */
  double a, b;                        /* a_num/a_den, b_num/b_den: one IEEE division each     */
} ceca_round_t;

/*
 * Host function.  The CECA schedule of iteration k:
 *   round      (out, may be NULL)  the scalars above;
 *   recv_from  (out, host, int32[n], may be NULL)  agent i receives the message of recv_from[i];
 *   send_to    (out, host, int32[n], may be NULL)  agent i sends its message to send_to[i].
 * recv_from is the row-to-column map of the permutation matrix P^(k) = Q^(r):
 *   CECA-2P, Eq. (2p-gossip-matrix-d1/d0): recv_from[i] = (i - n_r - delta_r) mod n;
 *   CECA-1P, Eq. (1p-gossip-matrix): even row i <-> row (i + 2 n_r + 1) mod n.
 * Errors: CECA_ERR_INVALID_ARG (n < 1, k < 0, bad variant), CECA_ERR_ODD_N_1P.
 */
ceca_status_t ceca_schedule(int32_t n, ceca_variant_t variant, int64_t k, ceca_round_t *round,
                            int32_t *recv_from, int32_t *send_to);

/*
 * One DSGD-CECA iteration for all agents, Eq. (x-iter-dsgd) and Eq. (y-iter-dsgd):
 *   u_i   = z_i - gamma e_i                         (the message of agent i; never stored)
 *   x+_i  = a (x_i - gamma e_i) + (1 - a) u_{recv_from[i]}
 *   y+_i  = b (y_i - gamma e_i) + (1 - b) u_{recv_from[i]}
 * X, Y, G: device, n x d fp32, leading dimension ld.  G may be NULL (treated as zero: a pure
 * CECA round of Sec. 3.1 / 3.2).  Y may be NULL only when the round ignores it (r = 0, where
 * b = 0 and z = x).
 * X_out, Y_out: device, same shape and ld.  Distinct buffers (ping-pong), or X_out == X and/or
 * Y_out == Y (in place: every element is read and then written by the same thread).  A crossed
 * alias (X_out == Y, Y_out == X, an output equal to G, X_out == Y_out) is CECA_ERR_UNSUPPORTED;
 * partially overlapping buffers are not detected and give undefined results.
 * X-only form: when n is a power of two every delta_r is 1 (Sec. 3.1), every message is built from
 * x, and X never depends on Y (CECA-2P is then the one-peer exponential graph).  Passing Y == NULL
 * and Y_out == NULL runs just the x update: 12 bytes per agent-parameter instead of 20.  For any
 * other n this combination is CECA_ERR_INVALID_ARG.
 * Dead-y form: in the last round of a cycle (r = tau-1) the new y is never used, because round 0 has
 * b = 0 and builds its message from x (Algorithm 1 with n_0 = 0).  Passing Y_out == NULL there (with Y
 * given) skips that write: 16 bytes per agent-parameter; the caller's Y buffer keeps its old contents
 * until round 0 overwrites it.  Y_out == NULL with Y given in any other round is CECA_ERR_INVALID_ARG.
 * fp32 arithmetic; a, b and 1-a, 1-b are formed in fp64 on the host and rounded once.
 * Speed: 128-bit accesses need ld % 4 == 0 and every array (X, Y, G, X_out, Y_out) starting the same
 * number of floats past a 16-byte boundary -- zero for whole allocations, or a common offset for
 * views that skip the same number of leading elements; up to three leading and three trailing
 * columns then run as a second, scalar launch.  Any other layout is correct too, but runs the scalar
 * form for every column (about 0.84 of the full rate).
 */
ceca_status_t ceca_gossip_sgd_step(const float *X, const float *Y, const float *G, float *X_out,
                                   float *Y_out, int32_t n, int64_t d, int64_t ld, float gamma,
                                   ceca_variant_t variant, int64_t k, void *stream);

/*
 * The same iteration with narrower storage (not in the paper, which only says that the update is
 * "additions and scaling"; the kernel is bound by the bytes it moves, so narrower storage is the
 * one way left to make it faster).  Arithmetic is fp32 in both forms; bf16 values are widened on
 * load and rounded to nearest even on store.
 *   xy_bf16 = 0: G is bf16 (n x d, leading dimension ld elements), X, Y, X_out, Y_out are fp32:
 *                18 bytes per agent-parameter instead of 20.  The result is the fp32 update of the
 *                gradient values as stored, to the same tolerance as ceca_gossip_sgd_step.
 *   xy_bf16 = 1: X, Y, G, X_out, Y_out are all bf16: 10 bytes per agent-parameter.  Every stored
 *                model value carries one bf16 rounding (relative 2^-9), so increments smaller than
 *                that are lost and the 1e-5 consensus accuracy of the fp32 form is out of reach:
 *                a bandwidth/accuracy trade the caller has to want.
 * Pointers are device pointers to fp32 or bf16 elements as stated; ld counts elements of either.
 * G and Y_out are required (no X-only or dead-y form); Y may be NULL where the round ignores it.
 * Full-width accesses need ld % 4 == 0 (xy_bf16 = 0) or ld % 8 == 0 (xy_bf16 = 1) and 16-byte
 * aligned fp32 / 8- resp. 16-byte aligned bf16 rows; anything else runs the scalar form.
 * Aliasing rules and error codes as for ceca_gossip_sgd_step.
 */
ceca_status_t ceca_gossip_sgd_step_bf16(const void *X, const void *Y, const void *G, void *X_out, void *Y_out,
                                        int32_t n, int64_t d, int64_t ld, int32_t xy_bf16, float gamma,
                                        ceca_variant_t variant, int64_t k, void *stream);

/*
 * `rounds` consecutive CECA rounds k0, k0+1, ..., k0+rounds-1 on (I, J) = (X, Y)
 * (Sec. 3.1 "Main recursions", Algorithm 2; Sec. 3.2 for the 1-port pairing).
 * After tau rounds that start at a multiple of tau every row of X_out is the column mean of
 * X and row i of Y_out is the mean of the other n-1 rows (Appendix B.2, Lemma "matrix
 * consensus"); one more round makes Y_out the mean as well.
 *
 *   fused = 0: one kernel launch per round, each a full pass over HBM.  Works for every n, d,
 *              ld and alignment.  Y_out == NULL is allowed when workspace holds n*ld floats, and
 *              without any workspace when n is a power of two (J then never feeds I).
 *   fused = 1 (CECA_FUSED_AUTO): a single launch.  A column tile of all n rows is brought on chip
 *              by TMA (cp.async.bulk.tensor), every round runs there, and the tile is written back
 *              once.  Three kernels exist and 1 picks by n and variant:
 *                4 (CECA_FUSED_BLOCK) keeps contiguous blocks of agents in registers, so that most of
 *                  the exchange is register to register and only block boundaries go through shared
 *                  memory; CECA-2P with 2 <= n <= 1152 (64-column tiles up to n = 150, 32-column tiles
 *                  up to n = 400, 16-column tiles above) and CECA-1P with n <= 416.  The fastest one
 *                  where it applies.
 *                2 (CECA_FUSED_SMEM) exchanges every row through shared memory; both variants,
 *                  n <= 2048 (32-column tiles up to n = 256, 8-column tiles above).  What 1 falls back
 *                  to beyond the limits of the first.
 *                3 (CECA_FUSED_TMEM) exchanges the rows through tensor memory (tcgen05.st /
 *                  tcgen05.ld); 2 <= n <= 128.  Kept for comparison; never picked by 1.
 *              Passing 2, 3 or 4 forces that kernel (CECA_ERR_UNSUPPORTED outside its range).
 *              All need X / X_out (and Y / Y_out when used) 16-byte aligned with ld*4 a multiple of
 *              16 (else CECA_ERR_ALIGNMENT), ld < 2^32 (more than 64 rounds run as several
 *              launches and then need Y_out), and a workspace of
 *              ceca_workspace_bytes(CECA_WS_CONSENSUS_FUSED, ...) bytes
 *              whose first int32 is a status word: it is left unchanged when the launch
 *              completes normally and set non-zero if a bounded on-chip wait for a TMA
 *              transfer ran out (read it with ceca_read_status); the tiles concerned are then
 *              not written.  Y may be NULL when the first round is r = 0; Y_out may be NULL.
 * X_out == X (and Y_out == Y) in place is allowed in every mode.
 */
typedef enum {
  CECA_UNFUSED = 0, CECA_FUSED_AUTO = 1, CECA_FUSED_SMEM = 2, CECA_FUSED_TMEM = 3, CECA_FUSED_BLOCK = 4
} ceca_fused_t;

ceca_status_t ceca_consensus_rounds(const float *X, const float *Y, float *X_out, float *Y_out,
                                    int32_t n, int64_t d, int64_t ld, ceca_variant_t variant,
                                    int64_t k0, int32_t rounds, int32_t fused, void *workspace,
                                    size_t workspace_bytes, void *stream);

/*
 * Per-agent logistic-regression gradient, the e^(k) of Algorithm 1 for the synthetic
 * classification workloads (the paper leaves f_i generic, Eq. (opt-problem-setting); this
 * particular loss is the benchmark's choice and has no counterpart in the paper):
 *   f_i(w)   = (1/m) sum_s log(1 + exp(-l_s <a_s, w>)),  l_s in {-1, +1}
 *   G[i, :]  = -(1/m) sum_s l_s sigma(-l_s <a_s, z_i>) a_s
 * evaluated at the model Algorithm 1 selects in iteration k: z = X if delta_r = 1, else Y.
 * A: device, n x m x d fp32, dense (sample rows contiguous, row stride d);
 * labels: device, n x m fp32 holding -1 or +1;  X, Y, G: device, n x d with leading dimension ld.
 * workspace: device, at least ceca_workspace_bytes(CECA_WS_LOGREG_GRAD, n, m, d) bytes; holds
 * per-block partial sums that a second, fixed-order pass adds up, so results are identical from
 * run to run.
 * Speed: A is read once when d % 4 == 0, ld % 4 == 0, d <= 65536 and A, X / Y, G are 16-byte aligned
 * (above d = 8192 the kernel runs as thread-block clusters, one column chunk per CTA); any other
 * shape is correct too but reads A twice (still with 128-bit loads when only d > 65536 stands in the way).
 */
ceca_status_t dsgd_logreg_grad(const float *A, const float *labels, const float *X, const float *Y,
                               int64_t k, float *G, int32_t n, int32_t m, int64_t d, int64_t ld,
                               ceca_variant_t variant, void *workspace, size_t workspace_bytes,
                               void *stream);

/*
 * Per-agent least-squares gradient, the paper's convex workload (Sec. 5 "DSGD: least-squares
 * problem"): f_i(w) = 1/2 ||A_i w - b_i||^2 and the stochastic gradient is
 *   G[i, :] = A_i^T (A_i z_i - b_i) + eps_i
 * evaluated at the model Algorithm 1 selects in iteration k (z = X if delta_r = 1, else Y).
 * A: device, n x m x d fp32, dense;  B: device, n x m fp32 (the measurements b_i);
 * noise: device, n x d with leading dimension ld, the caller's draw of eps (may be NULL = no noise);
 * X, Y, G, workspace, stream and the error codes: as for dsgd_logreg_grad (same workspace size).
 */
ceca_status_t dsgd_lsq_grad(const float *A, const float *B, const float *X, const float *Y, const float *noise,
                            int64_t k, float *G, int32_t n, int32_t m, int64_t d, int64_t ld,
                            ceca_variant_t variant, void *workspace, size_t workspace_bytes, void *stream);

/*
 * The gradient for a COLUMN SHARD (not in the paper, whose agents each own a whole model; this is the
 * form a deployment that splits the d parameter columns over several GPUs needs -- the gossip update
 * mixes rows only and needs no exchange between column blocks, the gradient needs one):
 *   1. dsgd_grad_shard_dots   dots[i, s] = <A_i[s, c0:c0+w], z_i[c0:c0+w]>        on every shard
 *   2. the sum of `dots` over the shards: an all-reduce of n x m floats between GPUs, or
 *      dsgd_grad_shard_sum (total = part when `first`, else total += part) called shard by shard
 *      where the shards share a GPU; a fixed order of additions makes the result reproducible
 *   3. dsgd_grad_shard_apply  turns the summed dots into the per-sample coefficients IN PLACE
 *      (loss = 0: -(1/m) l sigma(-l t) with targets = labels in {-1, +1}; loss = 1: t - b with
 *      targets = the measurements b) and writes G[:, c0:c0+w] = sum_s coef_s A_i[s, c0:c0+w] (+ noise)
 * A_shard: device, n x m x w with row stride lda >= w elements (lda = d when the shard is a view
 * of the full A, lda = w when it is stored on its own); Z_shard, G_shard, noise_shard: device,
 * n x w with leading dimensions ldz / ldg (the caller passes the block of X or of Y that
 * ceca_schedule's `payload` selects); dots: device, n x m.  No workspace.  The same error codes
 * as the other gradient calls.
 */
ceca_status_t dsgd_grad_shard_dots(const float *A_shard, const float *Z_shard, float *dots, int32_t n, int32_t m,
                                   int64_t w, int64_t lda, int64_t ldz, void *stream);
ceca_status_t dsgd_grad_shard_sum(float *total, const float *part, int64_t count, int32_t first, void *stream);
ceca_status_t dsgd_grad_shard_apply(const float *A_shard, const float *targets, float *dots, const float *noise_shard,
                                    float *G_shard, int32_t n, int32_t m, int64_t w, int64_t lda, int64_t ldg,
                                    int32_t loss, void *stream);

/*
 * dsgd_logreg_grad for callers that cannot provide a workspace because they cannot allocate device
 * memory when the gradient is needed: a plug-in inside an application that owns the device heap,
 * code running where a framework's allocator must not be re-entered, a latency-critical loop that
 * must stay clear of cudaMalloc.  (The paper has no counterpart to this call; it is a packaging
 * variant of the one above and computes exactly the same G with the same kernels.)
 *
 * The scratch memory is a fixed buffer of dsgd_logreg_grad_static_capacity() bytes (32 MiB) built
 * into the library; every GPU on which the library is used keeps that much memory from first use
 * until the process exits.  The call allocates nothing and frees nothing.
 *   - A problem whose ceca_workspace_bytes(CECA_WS_LOGREG_GRAD, n, m, d) exceeds the capacity is
 *     rejected with CECA_ERR_STATIC_SCRATCH before anything is launched.
 *   - The first call on each device looks up the buffer's device address (with that device
 *     current); make that first call ordinary eager work, before any stream capture is begun.
 *     The address is remembered per device ordinal for the life of the process: it does not
 *     survive cudaDeviceReset or the destruction of the device's primary context, after which
 *     this entry point must not be used again in the same process.
 *   - All calls on a device share the one buffer.  Nothing in it needs clearing between calls
 *     (each call overwrites what it later reads), but two calls that may run on the GPU at the
 *     same time -- different streams, or different host threads -- race on it: order them.
 * Arguments, layouts and the other error codes are those of dsgd_logreg_grad.
 */
ceca_status_t dsgd_logreg_grad_static(const float *A, const float *labels, const float *X, const float *Y,
                                      int64_t k, float *G, int32_t n, int32_t m, int64_t d, int64_t ld,
                                      ceca_variant_t variant, void *stream);

/* Host function.  Size in bytes of the buffer dsgd_logreg_grad_static works in. */
size_t dsgd_logreg_grad_static_capacity(void);

typedef enum {
  CECA_WS_CONSENSUS_FUSED = 1,    /* ceca_consensus_rounds, fused = 1                      */
  CECA_WS_CONSENSUS_UNFUSED = 2,  /* ceca_consensus_rounds, fused = 0 with Y_out == NULL   */
  CECA_WS_LOGREG_GRAD = 3,        /* dsgd_logreg_grad and dsgd_lsq_grad                    */
  CECA_WS_STEP_HOST = 4           /* ceca_gossip_sgd_step_host: the smallest useful size   */
} ceca_workspace_kind_t;

/* Host function.  Minimum workspace size in bytes for the call named by `kind`
 * (m is ignored except for CECA_WS_LOGREG_GRAD; pass ld for d where rows are padded). */
size_t ceca_workspace_bytes(ceca_workspace_kind_t kind, int32_t n, int32_t m, int64_t d);

/*
 * Host function.  Waits for `stream`, then copies the int32 status word at the start of a
 * fused-consensus workspace into *status_out (0 = no bounded wait ran out).  Zero the word
 * (cudaMemsetAsync) before the first launch that uses the workspace.
 */
ceca_status_t ceca_read_status(const void *workspace, int32_t *status_out, void *stream);

/*
 * Self-test of the bounded on-chip wait (no counterpart in the paper; meant for test suites, not for
 * production calls).  Launches the fused consensus kernel named by `fused` (CECA_FUSED_SMEM or
 * CECA_FUSED_TMEM) for one CECA-2P round on X, with the barrier that guards the TMA landing armed for
 * 16 bytes more than the transfer delivers and a poll budget of a few thousand polls.  The
 * transfer itself completes normally and nothing stays in flight; only the wait cannot succeed, so
 * every tile gives up: the status word at the start of `workspace` becomes non-zero and X_out
 * (which must not alias X) is left untouched.  Nothing traps; the context stays usable, and after
 * the word is cleared an ordinary call works as before.  Arguments as for ceca_consensus_rounds.
 */
ceca_status_t ceca_fused_wait_selftest(const float *X, float *X_out, int32_t n, int64_t d, int64_t ld,
                                       int32_t fused, void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same iteration as ceca_gossip_sgd_step for callers whose data lives in HOST memory
 * (pinned memory gives full copy bandwidth; pageable memory works but is slower).
 * X, Y (updated in place) and G are host pointers, n x d with leading dimension ld.  Columns
 * never interact in the update, so the call cuts the columns into slabs, and for each slab
 * copies X, Y, G to the device, runs the step kernel in place and copies X, Y back, with the
 * copies and the kernels of neighbouring slabs overlapping on internal streams.
 * workspace: DEVICE memory, workspace_bytes >= ceca_workspace_bytes(CECA_WS_STEP_HOST, n, 0, d);
 * more workspace means wider slabs.  The call returns after all slabs have been written back.
 * It takes no stream: the copies and kernels run on three internal non-blocking streams that are
 * created and destroyed inside the call and are ordered after nothing of the caller's.  Device work
 * of the caller that still reads or writes `workspace` (a pending kernel or memset on any stream)
 * must therefore have finished before the call; the host buffers must not be in use by pending copies.
 */
ceca_status_t ceca_gossip_sgd_step_host(float *X, float *Y, const float *G, int32_t n, int64_t d,
                                        int64_t ld, float gamma, ceca_variant_t variant, int64_t k,
                                        void *workspace, size_t workspace_bytes);

/* Host function.  A short English name for a status code (static storage). */
const char *ceca_status_string(ceca_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* CECA_H_ */
