/*
 * sd_verify.h -- C ABI of the verify-and-feedback step of speculative decoding
 * with an online-learned draft model (OnlineSpec, Algorithm 1).
 *
 * One call processes one decoding round for a batch of B sequences, each with k
 * draft tokens and a vocabulary of V entries:
 *
 *   p_{b,i} = softmax(T[b,i,:] / tau), i = 0..k   ("predicted distribution" of the
 *   q_{b,i} = softmax(D[b,i,:] / tau), i = 0..k-1   target / draft, Algorithm 1 inputs)
 *   accept draft token i  iff  u[b,i] < min(1, p_{b,i}(x_{b,i}) / q_{b,i}(x_{b,i}))
 *                                        (Algorithm 1, "Determine the accepted token length";
 *                                         the accept-iff form is restated in the proof of Lemma 1)
 *   n_b = index of the first rejected draft token, k if none
 *   y_b ~ max(0, p_{b,n_b} - q_{b,n_b}) normalised   if n_b < k
 *   y_b ~ p_{b,k}                                    if n_b = k
 *                                        (Algorithm 1, "Verify and update the draft sequence");
 *         drawn by inverse CDF in ascending vocabulary order with u[b,k]:
 *         y_b = min{ v : sum_{w<=v} r_w > u[b,k] * sum_w r_w }
 *   loss[b,i]   = KL(p_{b,i} || q_{b,i})                 (Eq. "kl_divergence" in the proof of
 *                 Lemma 1: the excess of the cross-entropy loss of Assumption 1 over its optimum)
 *   grad[b,i,v] = d loss[b,i] / d D[b,i,v] = (q_{b,i,v} - p_{b,i,v}) / tau
 *                                        (the feedback gradient "nabla f_t" of Sec. 3.1,
 *                                         taken w.r.t. the raw draft logits)
 *   acc_prob[b,i] = sum_v min(p, q) = 1 - TV(p, q)       (Eq. 1 and the proof of Lemma 1)
 *
 * Conventions common to every entry point
 *   - Unless an argument is documented as HOST, every pointer is a DEVICE pointer owned by the
 *     caller.  The library never frees or reallocates caller memory.
 *   - Tensors are dense, row-major, contiguous.  Logit rows may start at any element-aligned
 *     address; rows whose byte length and base address are multiples of 16 take the fast
 *     (bulk-copy, cluster) path, everything else takes a generic path with the same results
 *     that is about three times slower: pad the vocabulary to a multiple of 8 entries if you can.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = the legacy default
 *     stream).  The call does not synchronise; outputs are valid once the stream reaches the
 *     end of the enqueued work.
 *   - Return value: SD_OK, or a negative SD_ERR_* code for an error the host can detect; in that
 *     case nothing has been enqueued.  Problems only visible in the data on the device (a token
 *     outside [0,V), a row without a finite positive softmax denominator, a rejection whose
 *     residual is numerically zero) never trap: they set bits in out_status[b] and the affected
 *     outputs are memory-safe but otherwise unspecified.
 *   - dtype: SD_DTYPE_F32 (float) or SD_DTYPE_BF16 (bfloat16 bit patterns in uint16_t) for both
 *     logit tensors and for out_grad_draft.  Arithmetic is fp32 per element with fp64 row
 *     scalars in both cases.
 *   - Calls that share a workspace must not overlap on the GPU.
 *   - The library changes no setting of the caller's CUDA context unless asked to: with option
 *     SD_OPT_L2_PERSIST_MIB > 0 (default 0) the first call on a device sets the context's limit
 *     cudaLimitPersistingL2CacheSize to that many MiB, inside which the lines that the fast path's
 *     first pass fetches with the L2 evict_last policy are held for its second pass.  Since the second
 *     pass walks a row pair backwards (last fetched, first re-read) the set-aside no longer pays on the
 *     workloads measured, and sizes above about 60 MiB cost a third of the throughput.  See
 *     sd_set_option for the other tuning options; none is ever needed for correctness.
 */
#ifndef SD_VERIFY_H
#define SD_VERIFY_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SD_VERSION 100 /* major*10000 + minor*100 + patch */

/* dtype codes */
#define SD_DTYPE_F32 0
#define SD_DTYPE_BF16 1

/* return codes */
#define SD_OK 0
#define SD_ERR_NULL (-1)        /* a required pointer is NULL */
#define SD_ERR_SHAPE (-2)       /* B, k or V < 1, k > SD_MAX_K, or B*(k+1)*V overflows 2^62 */
#define SD_ERR_TEMPERATURE (-3) /* temperature is not a finite number > 0 */
#define SD_ERR_WORKSPACE (-4)   /* workspace NULL, misaligned (256 B) or too small */
#define SD_ERR_DTYPE (-5)       /* unknown dtype code */
#define SD_ERR_CUDA (-6)        /* a CUDA runtime call failed; text via sd_last_cuda_error() */
#define SD_ERR_NO_DEVICE (-7)   /* no sm_100 device is current */
#define SD_ERR_ALIGN (-8)       /* a pointer is not aligned to its element type */

#define SD_MAX_K 64 /* largest number of draft tokens per sequence */
#define SD_MAX_LEARNERS 8 /* largest number of draft models of an online ensemble */
#define SD_ENSEMBLE_SCRATCH_BYTES 256 /* device scratch of sd_ensemble_feedback */

/* bits of out_status[b] */
#define SD_STATUS_BAD_TOKEN 1u      /* some draft token of the sequence is outside [0,V): treated as rejected */
#define SD_STATUS_BAD_ROW 2u        /* a softmax denominator of the sequence is not finite and positive */
#define SD_STATUS_ZERO_RESIDUAL 4u  /* rejection with sum max(0,p-q) == 0: token drawn from p instead */
#define SD_STATUS_TIMEOUT 0x80000000u /* a bounded wait for a bulk copy gave up: outputs of the sequence are invalid */

/*
 * sd_verify_feedback / sd_verify_feedback_bf16 -- the whole step (Algorithm 1 from "Determine
 * the accepted token length" to "Receive interactive feedback") for fp32 / bf16 logits.
 *
 *   target_logits  [B, k+1, V]  in   row i < k pairs with draft row i; row k is the bonus row
 *   draft_logits   [B, k,   V]  in
 *   draft_tokens   [B, k]       in   int32, x[b,i] in [0,V)
 *   uniforms       [B, k+1]     in   fp32 in [0,1): u[b,0..k-1] drive the k accept tests,
 *                                    u[b,k] drives the residual / bonus draw
 *   temperature                 in   tau > 0, applied to both models' logits
 *   out_accept_len [B]          out  int32 n_b in [0,k]
 *   out_tokens     [B, k+1]     out  int32: x[b,0..n_b-1], then y_b at index n_b, then -1 padding
 *   out_loss       [B, k]       out  fp32 KL(p||q) per position; may be NULL together with
 *                                    out_grad_draft (verify-only mode)
 *   out_grad_draft [B, k, V]    out  (q-p)/tau, same dtype as the logits (bf16: round to nearest
 *                                    even); may be NULL (no gradient is written)
 *   stream                      in   cudaStream_t
 *
 * Scratch memory comes from a per-device buffer the library keeps and grows on demand
 * (cudaMalloc on the first call and whenever a larger problem arrives; that growth synchronises
 * the device).  Use sd_verify_feedback_ex to supply the scratch memory yourself.
 */
int sd_verify_feedback(const float* target_logits, const float* draft_logits,
                       const int32_t* draft_tokens, const float* uniforms, float temperature,
                       int B, int k, int V, int32_t* out_accept_len, int32_t* out_tokens,
                       float* out_loss, float* out_grad_draft, void* stream);

int sd_verify_feedback_bf16(const uint16_t* target_logits, const uint16_t* draft_logits,
                            const int32_t* draft_tokens, const float* uniforms, float temperature,
                            int B, int k, int V, int32_t* out_accept_len, int32_t* out_tokens,
                            float* out_loss, uint16_t* out_grad_draft, void* stream);

/*
 * sd_verify_feedback_ex -- same computation with every option exposed.
 *
 *   dtype            SD_DTYPE_F32 or SD_DTYPE_BF16; target_logits, draft_logits and out_grad_draft
 *                    are of that type
 *   workspace        device scratch of at least sd_workspace_bytes(B,k,V,dtype) bytes, aligned to
 *                    256 bytes; contents need not be initialised and are undefined afterwards
 *   out_acc_prob     [B,k] fp32 sum_v min(p,q) per position (Eq. 1), or NULL
 *   out_status       [B] uint32 SD_STATUS_* bits, or NULL
 */
int sd_verify_feedback_ex(const void* target_logits, const void* draft_logits,
                          const int32_t* draft_tokens, const float* uniforms, float temperature,
                          int B, int k, int V, int dtype, int32_t* out_accept_len,
                          int32_t* out_tokens, float* out_loss, void* out_grad_draft,
                          float* out_acc_prob, uint32_t* out_status, void* workspace,
                          size_t workspace_bytes, void* stream);

/*
 * sd_verify_feedback_hint -- sd_verify_feedback_ex plus the hint error of the optimistic online
 * update (Sec. 3.2, Eq. 3: the update looks ahead with a hint h_t, taken to be the last round's
 * gradient; Corollary 2 bounds the regret by the sum over rounds of ||h_t - grad f_t(w_t)||^2).
 * In the space of the draft logits, per position:
 *     out_hint_err[b,i] = sum_v ( hint[b,i,v] - (q_{b,i,v} - p_{b,i,v}) / tau )^2,
 * summed while the gradient is written: the hint is the only additional read (B*k*V entries).
 *   hint           in   [B,k,V] in `dtype`, the gradient a previous call wrote (or any tensor of that
 *                       shape); may be the same buffer as out_grad_draft -- every entry is read
 *                       before it is overwritten
 *   out_hint_err   out  [B,k] float; the difference is taken against the fp32 gradient before it is
 *                       rounded to `dtype`; partial sums in fp32 per warp, then fp64 in a fixed order
 *   workspace           at least sd_hint_workspace_bytes(B,k,V,dtype) bytes, 256-byte aligned
 * Everything else -- arguments, results, status bits, error codes -- as sd_verify_feedback_ex
 * (without out_acc_prob).  SD_ERR_NULL if hint or out_hint_err is NULL.
 */
size_t sd_hint_workspace_bytes(int B, int k, int V, int dtype);
int sd_verify_feedback_hint(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                            const float* uniforms, float temperature, int B, int k, int V, int dtype, const void* hint,
                            int32_t* out_accept_len, int32_t* out_tokens, float* out_loss, void* out_grad_draft,
                            float* out_hint_err, uint32_t* out_status, void* workspace, size_t workspace_bytes,
                            void* stream);

/*
 * sd_verify_feedback_static -- the same computation as sd_verify_feedback_ex for callers that
 * cannot allocate device memory.  (The paper has no counterpart of this entry point; it exists
 * for the way the library is embedded.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a serving loop whose
 * memory is handed out once at start-up by a pool that owns the whole device, in a process that
 * has been told to stay within a fixed footprint, or in a callback that may not call anything
 * that can synchronise the device or fail for lack of memory.  sd_verify_feedback allocates its
 * scratch on first use and sd_verify_feedback_ex wants a buffer from the caller; this entry point
 * needs neither, because its scratch is a fixed array of SD_STATIC_SCRATCH_BYTES bytes inside the
 * library itself.  The price: every GPU on which the library is loaded gives up that much memory
 * for as long as the process lives, whether this entry point is used or not.
 *
 * Arguments and results are those of sd_verify_feedback_ex without workspace/workspace_bytes.
 * It never calls cudaMalloc, cudaFree or any other allocating routine.  (The array itself becomes
 * resident when the CUDA runtime loads the library's device code on a GPU -- at the latest during
 * the first call of any entry point on that GPU -- not through a call of this function.)
 *
 *   - Shapes whose sd_workspace_bytes(B,k,V,dtype) exceeds SD_STATIC_SCRATCH_BYTES are refused
 *     with SD_ERR_WORKSPACE (sd_last_cuda_error() says how many bytes were needed); nothing is
 *     enqueued.  4 MiB covers, for instance, B*(k+1) up to about 1900 rows of fp32 logits (3800 of
 *     bf16) at V <= 131072.
 *   - The first call on each device looks up the device address of the array
 *     (cudaGetSymbolAddress, with that device current).  Make that first call outside any stream
 *     capture; later calls only enqueue a small memset and the kernel.
 *   - All calls on a device share the one array, and it keeps what the last call left in it.  The
 *     words that must start at zero are cleared on `stream` at the start of every call.  Two calls
 *     that overlap on the GPU (different streams without an ordering between them, or different
 *     host threads) race on the array and give wrong results: serialise them, or use
 *     sd_verify_feedback_ex with a scratch buffer per stream.
 */
#define SD_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
int sd_verify_feedback_static(const void* target_logits, const void* draft_logits,
                              const int32_t* draft_tokens, const float* uniforms, float temperature,
                              int B, int k, int V, int dtype, int32_t* out_accept_len,
                              int32_t* out_tokens, float* out_loss, void* out_grad_draft,
                              float* out_acc_prob, uint32_t* out_status, void* stream);

/* Bytes of scratch sd_verify_feedback_ex needs for this shape; 0 if the shape is invalid. */
size_t sd_workspace_bytes(int B, int k, int V, int dtype);

/*
 * sd_verify_greedy -- verification under greedy decoding: Algorithm 1 in the limit tau -> 0, the
 * decoding mode of the paper's experiments ("greedy decoding is adopted unless otherwise
 * specified", Sec. 4.1 Implementation Details).  The target distribution of a position is then
 * the point mass on its largest logit: a draft token is accepted iff it is the target's argmax of
 * its position, and the extra token is the target's argmax at the first mismatch, or at the bonus
 * position when everything was accepted.  No random numbers, no draft logits; only the target
 * logits are read, once.  (For the feedback loss of the same round call sd_verify_feedback_ex
 * with the temperature of the loss.)
 *
 *   target_logits  [B, k+1, V]  in   `dtype`; ties go to the smallest index; NaN entries are
 *                                    ignored; a row without an entry above -inf has argmax 0
 *   draft_tokens   [B, k]       in   int32; a token outside [0,V) simply matches nothing
 *   out_accept_len [B]          out  int32 n_b in [0,k]
 *   out_tokens     [B, k+1]     out  int32: x[b,0..n_b-1], argmax T[b,n_b,:] at index n_b, then -1
 *   out_argmax     [B, k+1]     out  int32 argmax of every target row, or NULL
 *   workspace                   in   device scratch of at least sd_greedy_workspace_bytes(B,k) bytes,
 *                                    aligned to 256 bytes, or NULL to use the library's own scratch
 *                                    (allocated and grown on demand, shared with sd_verify_feedback)
 *   stream                      in   cudaStream_t
 * Rows whose byte length and base address are multiples of 16 are read with 16-byte loads, all
 * others element by element.  Returns SD_OK or a negative SD_ERR_* code (nothing enqueued).
 */
int sd_verify_greedy(const void* target_logits, const int32_t* draft_tokens, int B, int k, int V,
                     int dtype, int32_t* out_accept_len, int32_t* out_tokens, int32_t* out_argmax,
                     void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of scratch sd_verify_greedy needs for this shape; 0 if the shape is invalid. */
size_t sd_greedy_workspace_bytes(int B, int k);

/*
 * sd_ensemble_feedback -- the feedback of one round for an online ensemble of N draft models
 * (Sec. 3.3, "Online Update with Ensemble"; N = 3 and epsilon = 10 in the paper's experiments).
 * Every base learner n gets the loss and the gradient of its own draft distribution
 * q^n = softmax(D^n/tau) against the same target distribution p = softmax(T/tau),
 *     loss[n,b,i] = KL(p_{b,i} || q^n_{b,i}),     grad^n[b,i,:] = (q^n_{b,i} - p_{b,i}) / tau,
 * each target row being fetched from HBM once for all N learners, and the meta learner's weights
 * follow the exponential weighting scheme  weight_n ~ exp(-epsilon * cumulative loss of learner n).
 * The loss of a round is the mean of the B*k per-position losses; out_cum_loss = cum_loss_in + that
 * mean, and out_weights are the weights of the NEXT round, computed from out_cum_loss.  Nothing is
 * verified or drawn here (use sd_verify_feedback / sd_verify_greedy with the logits of the combined
 * draft for that); the bonus rows of target_logits are not read.
 *
 *   target_logits   [B, k+1, V]   in   device, `dtype`
 *   draft_logits    [N]           in   HOST array of N device pointers, each [B, k, V] in `dtype`
 *   n_learners                    in   N, 1 .. SD_MAX_LEARNERS
 *   temperature, epsilon          in   tau > 0; epsilon >= 0 (SD_ERR_TEMPERATURE otherwise)
 *   cum_loss_in     [N] double    in   device, cumulative losses before this round, or NULL for zeros
 *   out_loss        [N, B, k]     out  device fp32
 *   out_grad        [N]           in   HOST array of N device pointers, each [B, k, V] in `dtype`
 *                                      (an entry may be NULL: no gradient for that learner), or NULL
 *   out_round_loss  [N] double    out  device, mean loss of the round per learner
 *   out_cum_loss    [N] double    out  device; may be the same buffer as cum_loss_in
 *   out_weights     [N] float     out  device, sums to 1
 *   out_status      [B] uint32    out  device SD_STATUS_BAD_ROW / SD_STATUS_TIMEOUT bits, or NULL
 *   workspace                     in   device scratch of SD_ENSEMBLE_SCRATCH_BYTES, aligned to 256
 *                                      bytes, or NULL for the library's own
 *   stream                        in   cudaStream_t
 * Rows must be whole 16-byte vectors and every tensor 16-byte aligned (SD_ERR_ALIGN otherwise:
 * there is no element-wise path for this entry point).  Two kernels are enqueued: the streaming
 * kernel of sd_verify_feedback over (sequence, row, learner) units, then a one-block reduction.
 */
int sd_ensemble_feedback(const void* target_logits, const void* const* draft_logits, int n_learners,
                         float temperature, float epsilon, int B, int k, int V, int dtype,
                         const double* cum_loss_in, float* out_loss, void* const* out_grad,
                         double* out_round_loss, double* out_cum_loss, float* out_weights,
                         uint32_t* out_status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * sd_verify_error_feedback -- the step with the feedback restricted to the error position, the
 * signal OSD collects (Sec. 3.1, "Online Update with Gradient Descent": the token positions where
 * the draft model was wrong, with the target's logits there, for a distillation loss on these
 * errors).  Verification is that of sd_verify_feedback, bit for bit: accept lengths and emitted
 * tokens are the same.  Of the gradient only the row of the first rejected position n_b of every
 * sequence is produced,
 *     out_error_grad[b, :] = (q_{b,n_b} - p_{b,n_b}) / tau      if n_b < k,      0 otherwise,
 * so the position it belongs to is out_accept_len[b].  The losses of all k positions are still
 * returned (the rejection tests need every row's softmax sums anyway).  Compared with the full step
 * the second pass runs over one row per sequence instead of k+1 and B*V instead of B*k*V gradient
 * entries are written.
 *
 *   target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, dtype,
 *   out_accept_len, out_tokens, out_loss (or NULL), out_status (or NULL): as in sd_verify_feedback_ex
 *   out_error_grad  [B, V]   out  `dtype`, or NULL
 *   workspace                in   device scratch of at least sd_workspace_bytes(B,k,V,dtype) bytes,
 *                                 aligned to 256 bytes, or NULL for the library's own
 * Rows must be whole 16-byte vectors and every tensor 16-byte aligned (SD_ERR_ALIGN otherwise: there
 * is no element-wise path for this entry point).  Two kernels are enqueued.
 */
int sd_verify_error_feedback(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                             const float* uniforms, float temperature, int B, int k, int V, int dtype,
                             int32_t* out_accept_len, int32_t* out_tokens, float* out_loss,
                             void* out_error_grad, uint32_t* out_status, void* workspace,
                             size_t workspace_bytes, void* stream);

/*
 * Vocabulary-parallel step -- the step of sd_verify_feedback for logits that are sharded along the
 * vocabulary, as a tensor-parallel output layer leaves them (the paper's deployment spreads a model
 * over four GPUs, Sec. 4.1 "Implementation Details").  Rank g of G holds the columns
 * [v_offset, v_offset + V_shard) of every row of both logit tensors; draft tokens, uniforms and
 * temperature are the same on every rank.  A softmax needs every column, so the step is three local
 * calls with an exchange after each; the library makes no collective call itself -- the caller
 * gathers with NCCL (or, on one GPU, by concatenation: no call waits for another rank).
 *
 *   sd_vp_partial   phase 1: per row the shard's softmax sums and, where the shard holds it, the
 *                   logits of the drafted token: out_records [B*(k+1)] records of SD_VP_RECORD_BYTES.
 *   exchange        all-gather the records: all_records [G][B*(k+1)], in rank order.
 *   sd_vp_finish    phase 2: merges the records (same bits on every rank), then out_accept_len [B],
 *                   out_loss [B,k] (or NULL), out_status [B] (or NULL) -- identical on every rank --,
 *                   the shard's columns of the gradient out_grad_shard [B,k,V_shard] (or NULL), and
 *                   out_local_mass [B][2] (double): the shard's share of the mass of the distribution the
 *                   extra token is drawn from (residual of row n_b, or the bonus row), and of the mass of
 *                   p_{n_b} (what a residual without mass falls back to).
 *   exchange        all-gather the shares: all_masses [G][B][2], in rank order.
 *   sd_vp_draw      phase 3: out_tokens [B,k+1]: the accepted draft tokens, then the extra token if this
 *                   rank's shard holds it (global index) and -1 otherwise, then -1 padding.
 *   exchange        element-wise maximum of out_tokens over the ranks.
 *
 * The same workspace (sd_vp_workspace_bytes, 256-byte aligned) must be passed to all three calls of
 * a round; it carries the row constants and region masses from phase 2 to phase 3.  Cuts must fall on
 * 16-byte boundaries (V_shard * element size a multiple of 16, shards 16-byte aligned): SD_ERR_ALIGN
 * otherwise.  Shards may differ in width.  A rejection whose residual has no mass on any rank (only a
 * forced rejection with q = p produces one) sets SD_STATUS_ZERO_RESIDUAL and draws from p_{n_b} instead,
 * as sd_verify_feedback does.
 * Every logit is read from HBM twice (once per phase).
 */
#define SD_VP_RECORD_BYTES 48
size_t sd_vp_workspace_bytes(int B, int k, int V_shard, int dtype);
int sd_vp_partial(const void* target_shard, const void* draft_shard, const int32_t* draft_tokens, float temperature,
                  int B, int k, int V_shard, int v_offset, int V_total, int dtype, void* out_records, void* workspace,
                  size_t workspace_bytes, void* stream);
int sd_vp_finish(const void* target_shard, const void* draft_shard, const int32_t* draft_tokens, const float* uniforms,
                 float temperature, int B, int k, int V_shard, int v_offset, int V_total, int dtype,
                 const void* all_records, int n_ranks, int rank, int32_t* out_accept_len, float* out_loss,
                 void* out_grad_shard, double* out_local_mass, uint32_t* out_status, void* workspace,
                 size_t workspace_bytes, void* stream);
int sd_vp_draw(const void* target_shard, const void* draft_shard, const int32_t* draft_tokens, const float* uniforms,
               float temperature, int B, int k, int V_shard, int v_offset, int V_total, int dtype,
               const int32_t* accept_len, const double* all_masses, int n_ranks, int rank, int32_t* out_tokens,
               uint32_t* out_status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * sd_bounds_report -- for the checked build of the library (compiled with -DSD_BOUNDS_CHECK: every index
 * the kernels form into global memory is tested against its extent before the access, an access that
 * fails is skipped and counted).  Waits for the current device, then fills out4 (host memory) with: the
 * number of violations since the last report, and the site code, index and limit of the first; the
 * counters go back to zero.  The regular build has no checks and reports out4[0] = 2^64 - 1.
 * Returns SD_OK, SD_ERR_NULL or SD_ERR_CUDA.
 */
int sd_bounds_report(unsigned long long* out4);

/*
 * sd_lmhead_grad -- the step after the feedback: the gradient of the round's loss with respect to
 * the weights W [V,d] of the draft model's linear output layer.  The feedback gradient of Sec. 3.1
 * ("nabla f_t(w_t)") reaches the parameters through the chain rule; with draft logits
 * D[r,:] = W x_r for the R = B*k positions of the round, and g = out_grad_draft of the step viewed
 * as [R,V],
 *     dW[v,j] = sum_r g[r,v] * x[r,j]                      (dW = g^T X).
 * (The paper leaves the draft network abstract; a linear output layer is what its draft heads end in.)
 * A dense contraction over the positions: tensor cores (tcgen05.mma, bf16 x bf16 -> fp32).
 *
 *   grad_logits  [R, V]   in   device, bfloat16 bit patterns: out_grad_draft of sd_verify_feedback_bf16
 *   hidden       [R, d]   in   device, bfloat16 bit patterns
 *   out_dW       [V, d]   out  device, fp32
 *   out_status   [1]      out  device uint32, or NULL: non-zero if a bounded wait inside the kernel gave
 *                              up (out_dW is then invalid)
 *   stream                in   cudaStream_t
 * V and d must be multiples of 8 and every pointer 16-byte aligned (SD_ERR_ALIGN otherwise); all
 * three tensors must be memory of the current GPU.  Returns SD_OK or a negative SD_ERR_* code
 * (nothing enqueued).
 */
int sd_lmhead_grad(const uint16_t* grad_logits, const uint16_t* hidden, int R, int V, int d, float* out_dW,
                   uint32_t* out_status, void* stream);

/*
 * sd_verify_feedback_host -- the same step for callers whose tensors live in HOST memory.
 * Every pointer is a HOST pointer (pinned memory gives asynchronous copies, pageable memory
 * works too).  The call copies the inputs to device buffers the library keeps per device
 * (grown on demand), runs the step in slices of sequences so that copies in both directions
 * overlap the kernels, copies every requested output back and returns after all of it has
 * completed.  out_loss, out_grad_draft, out_acc_prob and out_status may be NULL.
 */
int sd_verify_feedback_host(const void* target_logits, const void* draft_logits,
                            const int32_t* draft_tokens, const float* uniforms, float temperature,
                            int B, int k, int V, int dtype, int32_t* out_accept_len,
                            int32_t* out_tokens, float* out_loss, void* out_grad_draft,
                            float* out_acc_prob, uint32_t* out_status);

/*
 * Tuning options.  Each has a default, which an environment variable of the process (read once,
 * at the first use of the library) replaces, and which sd_set_option replaces at any time; a
 * change applies to the calls made after it.  Results never depend on them beyond rounding
 * (sums are taken in another order when the launch shape changes).
 *   SD_OPT_L2_PERSIST_MIB        env SD_VERIFY_L2_PERSIST_MIB   default 0    L2 set-aside requested on the
 *                                first call on a device; 0 = leave the context's limit untouched
 *   SD_OPT_CLUSTER               env SD_VERIFY_CLUSTER          default 0    cluster size of the fast path
 *                                (1..8), 0 = chosen per shape
 *   SD_OPT_LAG                   env SD_VERIFY_LAG              default -1   stages of the next row pair
 *                                that go before the second pass over a row pair; -1 = all of them when a
 *                                cluster has at most eight row pairs to work on, none otherwise; -2 = all
 *                                in every other cluster, none in the rest
 *   SD_OPT_L2_BUDGET_MIB         env SD_VERIFY_L2_MIB           default 80   bytes of row pairs in flight
 *                                between their two passes that the launch shape may assume L2 holds
 *   SD_OPT_FORCE_GENERIC         env SD_VERIFY_FORCE_GENERIC    default 0    non-zero: element-wise path
 *                                even for aligned rows
 *   SD_OPT_GREEDY_BLOCKS_PER_SM  env SD_GREEDY_BLOCKS_PER_SM    default 4    resident blocks of sd_verify_greedy
 *   SD_OPT_WAIT_POLLS            env SD_VERIFY_WAIT_POLLS       default 2^21 polls after which a wait
 *                                inside the fast path gives up (the sequences concerned then carry
 *                                SD_STATUS_TIMEOUT); the wait also ends after about a second
 *   SD_OPT_PREFETCH              env SD_VERIFY_PREFETCH         default 0    non-zero: while a block is in
 *                                its second pass over a row pair it asks L2 to fetch the next row pair
 * sd_set_option returns SD_OK, or SD_ERR_SHAPE for an unknown option; sd_get_option returns the
 * value in force, or -1 for an unknown option.
 */
#define SD_OPT_L2_PERSIST_MIB 0
#define SD_OPT_CLUSTER 1
#define SD_OPT_LAG 2
#define SD_OPT_L2_BUDGET_MIB 3
#define SD_OPT_FORCE_GENERIC 4
#define SD_OPT_GREEDY_BLOCKS_PER_SM 5
#define SD_OPT_WAIT_POLLS 6
#define SD_OPT_PREFETCH 7
#define SD_OPT_COUNT 8
int sd_set_option(int option_id, long long value);
long long sd_get_option(int option_id);

/*
 * sd_launch_info -- HOST out-parameters describing how the last successful device call on this
 * thread was launched: path (0 = generic, 1 = stream fast path, 2 = greedy verification, 3 = ensemble feedback, 4 = error-position feedback, 5 = output-layer gradient, 6 = vocabulary-parallel step), cluster size, threads per
 * block, dynamic shared memory per block, blocks launched, kernels launched.  Any pointer may
 * be NULL.  Diagnostic only.
 */
void sd_launch_info(int* path, int* cluster_size, int* threads, int* smem_bytes, int* blocks,
                    int* kernels);

/* Release the per-device scratch and staging buffers the library keeps (synchronises). */
void sd_release_cached_buffers(void);

/* Text for a return code; never NULL. */
const char* sd_strerror(int code);

/* Text of the CUDA error behind the last SD_ERR_CUDA on this thread ("" if none). */
const char* sd_last_cuda_error(void);

/* SD_VERSION of the loaded library. */
int sd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SD_VERIFY_H */
