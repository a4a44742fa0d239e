/*
 * kdkl - fused chunked KL distillation loss for NVIDIA B200 (sm_100a), C ABI.
 *
 * The loss is the forward KL divergence between a cached top-K teacher and the student's
 * softmax over the LM head, evaluated with the output projection fused into the loss so the
 * [T, V] logit tensor never exists (paper, section "Full Chunked KL Computation",
 * Algorithm 1). Per token, with z = W h the student logits, q = softmax(z / tau), p the teacher
 * probabilities on the support S (|S| = K), M = sum_S p the retained mass (not renormalised):
 *
 *     L = sum_S p log p  -  sum_S p z / tau  +  M log Z          (Eq. "decomp")
 *     dL/dz_v = (M q_v - p_v) / tau                              (Eq. "grad"; 1/tau = chain rule)
 *
 * and the reported loss is the mean of L over the tokens whose mask is 1 (text under Eq. "kl").
 *
 * Conventions for every entry point unless stated otherwise
 *   - all data pointers are DEVICE pointers owned by the caller; the library allocates no
 *     device memory and only enqueues work on the given stream (no host synchronisation).
 *     Between calls it keeps nothing of a call's data: its only state is, per thread, the text of
 *     the last error and the last launch count, and, per process, what it has learnt about each
 *     device (SM count, compute capability, kernel attributes already set) plus the test hook
 *     kdkl_debug_guard_bytes;
 *   - matrices are row-major and contiguous; hidden, weight and the workspace must be
 *     16-byte aligned; H must be a multiple of 8;
 *   - return value: KDKL_OK or a negative KDKL_ERR_* detected on the host before anything
 *     was enqueued (outputs untouched). Conditions only the device can see are recorded in
 *     the workspace and read with kdkl_status().
 */
#ifndef KDKL_H_
#define KDKL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KDKL_OK 0
#define KDKL_ERR_NULL (-1)      /* a required pointer is NULL */
#define KDKL_ERR_SHAPE (-2)     /* T, H, V, K < 1; K > KDKL_MAX_K; H % 8 != 0; V >= 2^31 */
#define KDKL_ERR_ALIGN (-3)     /* hidden / weight / workspace / outputs not 16-byte aligned */
#define KDKL_ERR_WORKSPACE (-4) /* workspace smaller than kdkl_workspace_bytes() */
#define KDKL_ERR_ARG (-5)       /* temperature <= 0, chunk < 0, bad option value */
#define KDKL_ERR_ARCH (-6)      /* current device is not compute capability 10.x */
#define KDKL_ERR_CUDA (-7)      /* a CUDA call failed; kdkl_last_error() has the text */
/* device-detected, reported by kdkl_status(): */
#define KDKL_ERR_TIMEOUT (-8)   /* a bounded wait inside a kernel expired */
#define KDKL_ERR_STATE (-9)     /* backward called on a workspace forward did not fill for this shape, chunk size and
                                   temperature (or, with stored_exponentials, whose exponentials are gone) */
#define KDKL_ERR_INDEX (-10)    /* a teacher index >= V was seen (the entry was ignored) */
#define KDKL_ERR_NONFINITE (-11)/* a counted token's loss is not finite */
#define KDKL_ERR_RANGE (-13)    /* stored exponentials only (kdkl_forward_backward, option stored_exponentials): a
                                   counted token's scaled logits all lie below the range the bf16 exponentials
                                   keep (log2 of its normaliser < -40); use kdkl_forward + kdkl_backward there */

#define KDKL_MAX_K 1024

typedef struct kdkl_options {
  int32_t struct_size;        /* sizeof(kdkl_options), for versioning */
  int32_t teacher_mode;       /* 0: values are logits, p = exp(l/tau - Lambda), Lambda = teacher_lse[t] if given
                                    (retained mass M < 1 possible, as in the paper) else logsumexp over the
                                    row's K values (M = 1);
                                 1: values are log-probabilities, p = exp(l), tau must be 1 */
  int32_t accumulate_dweight; /* 0: dweight is overwritten; 1: dweight += */
  int32_t dhidden_dtype;      /* 0: bf16; 1: fp32 */
  float denom_override;       /* <= 0: mean over this call's counted tokens; > 0: divide by this instead */
  int32_t stored_exponentials;/* 1: only when one chunk covers all T tokens (chunk >= T): the forward call also
                                 leaves the bf16 exponentials 2^(z log2e / tau - 64) in the workspace's [T, V]
                                 buffer and kdkl_backward forms G from them instead of projecting again (three
                                 projections for the two calls, as in kdkl_forward_backward; the vocabulary-sharded
                                 calls included, where log Z is only known after the exchange). Otherwise
                                 KDKL_ERR_ARG. The conversion is in place, so kdkl_backward can run ONCE per
                                 forward call in this mode: a second one reports KDKL_ERR_STATE and writes nothing.
                                 A struct of the previous size (without this field) is accepted */
  const double* denom_device; /* NULL, or a DEVICE pointer to one double read when the kernels run: the divisor of
                                 the mean (takes precedence over denom_override). For data-parallel callers that
                                 sum kdkl_count_tokens over their ranks on the device: no host read of the count.
                                 A struct of a previous size (without this field) is accepted */
  int32_t dw_chunks_per_pass; /* 0 (default): with chunks of at most 4096 tokens, dweight += G^T h runs once per two
                                 chunks (the dlogits of both are kept: one more [chunk, V] bf16 buffer in the
                                 workspace, 1 GiB at chunk 4096 and V = 131072), which halves the fp32
                                 read-modify-write traffic of dweight; 1: once per chunk, without that buffer;
                                 2: as 0. Measured on one B200 at T = 131072, H = 4096, V = 131072: 413-416 ms with
                                 8.15 GB peak (default) against 415-420 ms with 7.07 GB (1); at chunk 2048,
                                 H = 3072: 74.9 against 77.0 ms. Same results up to fp32 reassociation in dweight.
                                 kdkl_workspace_bytes must be given the same options as the calls.
                                 A struct of a previous size (without this field) is accepted */
  const float* grad_loss_device; /* NULL, or a DEVICE pointer to one float read when the kernels run: the upstream
                                 gradient dL_total/dloss, in place of the grad_loss argument of kdkl_backward,
                                 kdkl_forward_backward and the host-record step (the argument is then ignored). For
                                 callers that hold the upstream gradient on the device (an autograd engine): no
                                 host read. A struct of a previous size (without this field) is accepted */
} kdkl_options;

/* Number of counted tokens of a batch (mask = 1; T when loss_mask is NULL), written as one double to
 * count_out (DEVICE). One small kernel on the stream. The divisor of the mean for a caller whose tokens
 * are spread over several ranks is the sum of these counts (text under Eq. "kl": the mean runs over all
 * loss-masked positions); pass that sum back through kdkl_options.denom_device. */
int kdkl_count_tokens(const uint8_t* loss_mask, int64_t T, double* count_out, void* cuda_stream);

/* Bytes of device workspace forward and backward need for this shape (chunk 0 = default 4096).
 * The same workspace must be passed to forward and then to backward: it carries the saved
 * state of Algorithm 1 (log Z, M, the prepared teacher) and the transient per-chunk buffers. */
size_t kdkl_workspace_bytes(int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk,
                            const kdkl_options* opt);

/* Debug aids for tests (no counterpart in the paper). kdkl_workspace_layout: the table of the workspace's slabs, in
 * layout order, as byte offsets and used lengths; returns the number of slabs (fills at most `capacity` entries).
 * kdkl_debug_guard_bytes(n): from now on (process-wide, until changed; n = 0 restores the compact layout, n is
 * rounded up to 256 and capped at 1 MiB) every layout leaves n untouched bytes after every slab, so a test can
 * pre-fill the workspace, run, and check that nothing wrote past the end of a slab; returns the previous value. */
int kdkl_workspace_layout(int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, const kdkl_options* opt,
                          int64_t* offsets, int64_t* lengths, int32_t capacity);
int64_t kdkl_debug_guard_bytes(int64_t n);

/* Forward (Algorithm 1, "Forward"; Eq. "decomp"). One tensor-core sweep per chunk computes the
 * online max / sum-exp over the vocabulary and gathers z at the teacher's indices.
 *   hidden_bf16   [T, H]  bf16   student final hidden states
 *   weight_bf16   [V, H]  bf16   LM-head weight
 *   topk_idx      [T, K]  int32  teacher support; < 0 = empty slot; >= V = ignored + KDKL_ERR_INDEX;
 *                                duplicates within a row add
 *   topk_val      [T, K]  fp32   teacher values (see teacher_mode)
 *   teacher_lse   [T] fp32 or NULL   full-vocabulary teacher logsumexp at temperature tau
 *   loss_mask     [T] uint8 or NULL  1 = counted, 0 = ignored (teacher row is never read). Row tiles
 *                                (256 consecutive tokens of a chunk) without a counted token are skipped
 *                                by every tensor-core sweep, forward and backward: padding costs nothing
 *   chunk         tokens per chunk, 0 = default; the result does not depend on it
 *   loss_out      [1] fp32  mean loss
 *   loss_per_token [T] fp32 or NULL  (0 at ignored tokens)
 *   gathered_logits [T, K] fp32 or NULL  z at topk_idx, caller's slot order (NaN where not gathered)
 *   gathered_idx  [T, K] int32 or NULL   the vocabulary column the kernel read for each slot (-1 where none)
 */
int kdkl_forward(const void* hidden_bf16, const void* weight_bf16, const int32_t* topk_idx,
                 const float* topk_val, const float* teacher_lse, const uint8_t* loss_mask,
                 int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, float temperature,
                 const kdkl_options* opt, void* workspace, size_t workspace_bytes,
                 float* loss_out, float* loss_per_token, float* gathered_logits,
                 int32_t* gathered_idx, void* cuda_stream);

/* Backward (Algorithm 1, "Backward"; Eq. "grad"). Per chunk: recompute the logit tile in tensor
 * memory, form G = (M q - p) g / tau in registers, then dhidden = G W and dweight += G^T h.
 * Same hidden / weight / mask / shape / chunk / temperature / opt as the forward call, and the
 * workspace that call filled.
 *   grad_loss  d(total)/d(loss_out), usually 1 (ignored when kdkl_options.grad_loss_device is set)
 *   dhidden    [T, H] bf16 (or fp32, see options); rows of ignored tokens are exact zeros
 *   dweight    [V, H] fp32
 */
int kdkl_backward(const void* hidden_bf16, const void* weight_bf16, const uint8_t* loss_mask,
                  int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, float temperature,
                  const kdkl_options* opt, float grad_loss, void* workspace, size_t workspace_bytes,
                  void* dhidden, float* dweight, void* cuda_stream);

/* Forward and backward in one call, with three projections instead of four. The paper's backward recomputes
 * each chunk's logits (Algorithm 1, "Backward": a second output projection) because it runs as a separate
 * autograd phase; when the gradient is wanted right away - the loss is the last operation of a training step -
 * the forward sweep of a chunk can leave the unnormalised exponentials e = 2^(z log2e / tau - 64) in the chunk's
 * [chunk, V] bf16 buffer. As soon as the chunk's log Z is known, G = (M q - p) g / tau (Eq. "grad") is
 * s_t e - b_t p with one scale s_t per token, and that scale is taken out of the two contractions instead of being
 * written into the buffer: dhidden rows are multiplied by it in fp32, dweight is contracted against hidden rows
 * scaled by it (rounded to bf16), and only the <= K teacher entries of a row are patched in place. Same workspace
 * size class, same outputs as kdkl_forward followed by kdkl_backward up to two more bf16 roundings (the stored
 * exponential; for dweight also the scaled hidden rows). Limits of the stored exponential: a scaled logit
 * z log2e / tau beyond +192 cannot be stored (kdkl_status: KDKL_ERR_NONFINITE with the token), and a token whose log2
 * normaliser is below -40 would lose entries to underflow (KDKL_ERR_RANGE); use the two-call path for such inputs.
 * 6 T H V flops instead of 8 T H V.
 * Arguments as the two calls; grad_loss must be known here. The workspace afterwards holds the same saved
 * state (kdkl_saved_state, kdkl_status). Vocabulary shards need the cross-shard exchange before log Z is known:
 * there the same saving is available through option stored_exponentials when one chunk covers all tokens. */
int kdkl_forward_backward(const void* hidden_bf16, const void* weight_bf16, const int32_t* topk_idx,
                          const float* topk_val, const float* teacher_lse, const uint8_t* loss_mask, int64_t T,
                          int64_t H, int64_t V, int32_t K, int64_t chunk, float temperature, const kdkl_options* opt,
                          float grad_loss, void* workspace, size_t workspace_bytes, float* loss_out,
                          float* loss_per_token, void* dhidden, float* dweight, void* cuda_stream);

/* Vocabulary-sharded use (the paper's tensor-parallel variant: section "Full Chunked KL Computation", last
 * sentences, and Algorithm 1's "distributed max", "reduce sigma", "reduce dh across shards").
 * Rank r holds the weight rows [vocab_offset, vocab_offset + V_local) of a vocabulary of V_total entries;
 * hidden states, the teacher record (GLOBAL indices) and the mask are replicated. Per step and rank:
 *   1. kdkl_forward_shard: the local sweep. Writes shard_stats [2, T] fp32 (device): row 0 the local
 *      log2-domain normaliser log2 sum_{v local} 2^(z_v log2e / tau), row 1 the local cross term
 *      sum_{k local} p_k z_k / tau. M and the teacher entropy use all usable entries on every rank.
 *      gathered_logits / gathered_idx (optional) are filled for the local entries only (global index).
 *   2. the caller gathers the shard_stats of all ranks into all_stats [n_shards, 2, T] (for instance an
 *      NCCL all-gather); this library performs no communication.
 *   3. kdkl_forward_finish: log Z = logsumexp over shards, C = sum over shards, loss as in kdkl_forward;
 *      identical on every rank. Stores the global log Z in the workspace for backward.
 *   4. kdkl_backward with weight_local, V = V_local and the same workspace: dweight is the local slice
 *      [V_local, H] (complete, no communication); dhidden is this shard's partial sum over its vocabulary
 *      rows, to be summed over ranks by the caller (use dhidden_dtype = 1 for an fp32 reduction).
 * V_total < 2^30. Other arguments and errors as kdkl_forward. */
int kdkl_forward_shard(const void* hidden_bf16, const void* weight_local_bf16, const int32_t* topk_idx,
                       const float* topk_val, const float* teacher_lse, const uint8_t* loss_mask,
                       int64_t T, int64_t H, int64_t V_local, int64_t vocab_offset, int64_t V_total, int32_t K,
                       int64_t chunk, float temperature, const kdkl_options* opt, void* workspace,
                       size_t workspace_bytes, float* shard_stats, float* gathered_logits,
                       int32_t* gathered_idx, void* cuda_stream);
int kdkl_forward_finish(const float* all_stats, int32_t n_shards, const uint8_t* loss_mask, int64_t T, int64_t H,
                        int64_t V_local, int32_t K, int64_t chunk, float temperature, const kdkl_options* opt,
                        void* workspace, size_t workspace_bytes, float* loss_out, float* loss_per_token,
                        void* cuda_stream);

/* Synchronises the stream and reads the device status of the last forward/backward on this
 * workspace: *code = KDKL_OK or a device-detected KDKL_ERR_*; detail[0] = site/row of the error,
 * detail[1] = number of counted tokens, detail[2] = number of ignored (>= V) teacher indices.
 * detail may be NULL. */
int kdkl_status(const void* workspace, void* cuda_stream, int32_t* code, int64_t* detail);

/* Saved per-token scalars of Algorithm 1 inside a workspace forward has filled (device pointers
 * into the workspace; valid until the workspace is reused): log Z of z/tau and the retained mass M
 * (both 0 at ignored tokens). */
int kdkl_saved_state(void* workspace, int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk,
                     const kdkl_options* opt, const float** logZ, const float** mass);

/* Forward + backward with HOST buffers (the end-to-end call): copies the inputs to the device
 * arena, runs both passes, copies loss, dhidden and dweight back, and synchronises the stream.
 * Host pointers: hidden, weight, topk_idx, topk_val, teacher_lse (or NULL), loss_mask (or NULL),
 * loss_out [1], dhidden_out [T,H] (dtype per options), dweight_out [V,H] fp32 (either may be NULL
 * to skip that copy). device_arena is a device buffer of at least kdkl_host_arena_bytes().
 * With more than one chunk the call overlaps what it can with the chunk loop: the hidden rows of chunk i are
 * uploaded on a second stream (created and destroyed inside the call, like the events that order the two
 * streams; no device memory is allocated) while earlier chunks are swept, and the dhidden rows of chunk i are
 * downloaded while later chunks are differentiated; the weight, the teacher record and dweight, which the whole
 * step needs or produces, travel on the caller's stream. Use pinned host memory, or the copies serialise. */
size_t kdkl_host_arena_bytes(int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk,
                             const kdkl_options* opt);
int kdkl_forward_backward_host(const void* hidden_bf16, const void* weight_bf16, const int32_t* topk_idx,
                               const float* topk_val, const float* teacher_lse, const uint8_t* loss_mask,
                               int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, float temperature,
                               const kdkl_options* opt, float grad_loss, void* device_arena,
                               size_t arena_bytes, float* loss_out, void* dhidden_out, float* dweight_out,
                               void* cuda_stream);

/* One step the way the offline pipeline of the paper feeds it (section "Offline Distillation with a Top-K
 * Teacher": the teacher's top-K record is cached ahead of time and read back per batch): the record of this
 * batch - topk_idx, topk_val, optional teacher_lse, optional loss_mask - arrives from HOST memory (pinned for
 * full copy speed), while the student's hidden states, the head weight, both gradients and the workspace live
 * on the DEVICE, as they do inside a training loop. Copies the record into `staging` (device,
 * kdkl_record_staging_bytes(T, K) bytes, 256-byte aligned), runs kdkl_forward and kdkl_backward on the stream,
 * copies the loss to loss_out (HOST, 4 bytes) and synchronises the stream before returning. Errors as the
 * two calls; device-detected conditions through kdkl_status(workspace). */
size_t kdkl_record_staging_bytes(int64_t T, int32_t K);
int kdkl_step_host_record(const void* hidden_bf16, const void* weight_bf16, const int32_t* topk_idx_host,
                          const float* topk_val_host, const float* teacher_lse_host, const uint8_t* loss_mask_host,
                          int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, float temperature,
                          const kdkl_options* opt, float grad_loss, void* staging, size_t staging_bytes,
                          void* workspace, size_t workspace_bytes, float* loss_out_host, void* dhidden,
                          float* dweight, void* cuda_stream);

/* Forward + backward on DEVICE buffers with a CUDA event between every kernel; synchronises and
 * returns, per stage, the summed device time in ms and the number of launches. Stages:
 * 0 teacher prep, 1 forward GEMM + online log-sum-exp + gather, 2 partial combine, 3 loss reduce,
 * 4 backward coefficients, 5 recompute GEMM + dlogits, 6 dhidden GEMM, 7 dweight GEMM.
 * stage_ms and stage_launches are HOST arrays of 8. Arguments as kdkl_forward / kdkl_backward. */
int kdkl_profile_stages(const void* hidden_bf16, const void* weight_bf16, const int32_t* topk_idx,
                        const float* topk_val, const float* teacher_lse, const uint8_t* loss_mask,
                        int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, float temperature,
                        const kdkl_options* opt, float grad_loss, void* workspace, size_t workspace_bytes,
                        float* loss_out, void* dhidden, float* dweight, void* cuda_stream,
                        float* stage_ms, int32_t* stage_launches);

/* The tensor-core mainloop on its own: C[M,N] (fp32, row-major) = A * B^T with bf16 operands.
 * a_mn = 0: A is [M, K] row-major; 1: A is stored [K, M]. b_mn likewise for B ([N, K] or [K, N]).
 * M, N, K multiples of 8. status: device int32[2] the caller zeroed, receives {KDKL_ERR_TIMEOUT, site}
 * if a bounded wait expires, or NULL. Used to validate and time the GEMM under the fused epilogues. */
int kdkl_gemm_bf16(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K,
                   int32_t a_mn, int32_t b_mn, int32_t* status, void* cuda_stream);

/* (No counterpart in the paper: an addition for callers that cannot allocate device memory.)
 * log Z[t] = logsumexp over the vocabulary of (W h_t) / temperature, the normaliser of Eq. "decomp",
 * computed without any device allocation: the caller passes only inputs and the output, and the
 * scratch for the per-vocab-tile partials is a fixed array inside the library (about 8 MiB, held by
 * every GPU that loads the library until the process exits).
 * Meant for code that may not call cudaMalloc: a plugin inside a server whose memory pool already owns
 * the device, or a latency-critical callback that must stay out of the driver's allocator.
 *   hidden_bf16 [T, H], weight_bf16 [V, H], logz_out [T] fp32: device pointers; H % 8 == 0;
 *   V <= 262144 (larger V is rejected with KDKL_ERR_WORKSPACE and a message on stderr); any T >= 1
 *   (processed 1024 tokens at a time). No cudaMalloc / cudaFree / allocating library call is made.
 * The first call on each device also resolves the scratch array's device address and sets a kernel
 * attribute; make that first call before any stream capture is open. All calls share the one scratch
 * array and it keeps the previous call's contents (the parts that must start at zero are cleared on the
 * stream at the start of each call): calls that overlap on the same GPU, on any streams, race.
 * If a bounded wait inside the kernel expires, the affected outputs are NaN. */
int kdkl_logz_noalloc(const void* hidden_bf16, const void* weight_bf16, int64_t T, int64_t H, int64_t V,
                      float temperature, float* logz_out, void* cuda_stream);

#define KDKL_ERR_OVERFLOW (-12) /* teacher top-K: a row's candidate list still overflows after four rounds of a tightened
                                   threshold (in practice: hundreds of logits tied exactly at the K-th value) */

/* The teacher cache record of the offline pipeline (paper, section "Offline Distillation with a Top-K
 * Teacher": the K largest entries per position are cached; the retained mass M <= 1 is not renormalised,
 * which needs the full normaliser). For teacher hidden states [T, H] and teacher head [V, H] (bf16):
 *   topk_idx [T, K] int32, topk_val [T, K] fp32: the K largest logits z = W h per token, by value
 *            descending, ties by the smaller index first (exact selection, not an approximation);
 *   lse [T] fp32: log sum_v exp(z_v / temperature), the `teacher_lse` argument of kdkl_forward.
 * Two tensor-core sweeps: the first gives the log-sum-exp and per-vocab-tile maxima, whose K-th largest
 * is a threshold that every member of the top-K must reach; the second recomputes the logits and keeps
 * those at or above it; a per-row sort finishes. When large logits cluster in a few vocabulary tiles (a
 * frequency-ordered vocabulary), or the vocabulary has fewer than K tiles of 256 columns, more logits reach that
 * threshold than a row's candidate list holds (max(4 K, 256) slots, at most 1024; the whole vocabulary when
 * V <= 8192): the list then keeps a uniform sample of them, the K-th largest kept candidate serves as a tighter
 * threshold and the row is scanned again, up to four times (sweeps that no row needs return at once; each round
 * keeps about K / slots of the candidates). K <= 256, K <= V <= 2^20, H % 8 == 0.
 * workspace: device, kdkl_teacher_topk_workspace_bytes(); its first words are a status block readable
 * with kdkl_status (KDKL_ERR_OVERFLOW / KDKL_ERR_TIMEOUT). Enqueue-only. */
size_t kdkl_teacher_topk_workspace_bytes(int64_t T, int64_t H, int64_t V, int32_t K);
int kdkl_teacher_topk(const void* hidden_bf16, const void* weight_bf16, int64_t T, int64_t H, int64_t V, int32_t K,
                      float temperature, void* workspace, size_t workspace_bytes, int32_t* topk_idx,
                      float* topk_val, float* lse, void* cuda_stream);

/* The same per-stage measurement for kdkl_forward_backward. Stage 5 is then the in-place conversion of the stored
 * exponentials into G (the place of the recompute GEMM); the other stages as above. */
int kdkl_profile_single_pass(const void* hidden_bf16, const void* weight_bf16, const int32_t* topk_idx,
                             const float* topk_val, const float* teacher_lse, const uint8_t* loss_mask, int64_t T,
                             int64_t H, int64_t V, int32_t K, int64_t chunk, float temperature,
                             const kdkl_options* opt, float grad_loss, void* workspace, size_t workspace_bytes,
                             float* loss_out, void* dhidden, float* dweight, void* cuda_stream, float* stage_ms,
                             int32_t* stage_launches);

#define KDKL_FEATURE_MSE 0
#define KDKL_FEATURE_COSINE 1

/* Hidden-state feature loss that the paper recommends adding to the logit KL (section "Additional
 * Ablations", paragraph "Loss design": a mean-squared-error variant and a cosine variant; no formula is
 * printed, these are the textbook ones). Per token t, student row s and teacher row r of width H:
 *   KDKL_FEATURE_MSE     f_t = (1/H) sum_h (s_h - r_h)^2
 *   KDKL_FEATURE_COSINE  f_t = 1 - <s,r> / (|s| |r|)        (f_t = 1, zero gradient, when |s||r| <= 1e-12)
 *   loss = weight * sum_t mask_t f_t / N,  N = number of mask = 1 tokens (denom_override > 0 replaces it;
 *   N = 0 gives loss 0 and zero gradients), reduced in a fixed order (bitwise reproducible).
 * Loss and gradient come out of one pass over the inputs (the op is bound by memory traffic):
 *   dstudent_bf16 [T, H] or NULL = loss only: grad_loss * d loss / d student, rounded once to bf16;
 *     accumulate = 0 overwrites it (ignored tokens' rows are set to zero), accumulate = 1 adds to what it
 *     holds, e.g. the dHidden that kdkl_backward wrote for the same hidden states (ignored rows untouched).
 *   student_bf16, teacher_bf16 [T, H]: device, row-major, 16-byte aligned, H % 8 == 0; rows of ignored
 *     tokens are never read. loss_mask [T] u8 or NULL = all counted. loss_out [1], loss_per_token [T] or
 *     NULL (f_t, 0 on ignored tokens): device fp32. Must not alias one another.
 *   workspace: device, 16-byte aligned, kdkl_feature_loss_workspace_bytes(T). Enqueue-only, two kernels (three with a mask).
 * Returns KDKL_OK or KDKL_ERR_NULL / _SHAPE / _ARG (unknown kind, non-finite weight or grad_loss,
 * accumulate not 0/1) / _ALIGN / _WORKSPACE / _ARCH / _CUDA. */
size_t kdkl_feature_loss_workspace_bytes(int64_t T);
int kdkl_feature_loss(const void* student_bf16, const void* teacher_bf16, const uint8_t* loss_mask, int64_t T,
                      int64_t H, int32_t kind, float weight, float grad_loss, float denom_override,
                      int32_t accumulate, void* workspace, size_t workspace_bytes, float* loss_out,
                      float* loss_per_token, void* dstudent_bf16, void* cuda_stream);

/* kdkl_feature_loss with the upstream gradient read on the device when the kernels run (one float; for
 * callers such as an autograd engine that hold it there: no host read). Always three kernels. Otherwise as above;
 * KDKL_ERR_NULL when grad_loss_device is NULL. */
int kdkl_feature_loss_device_grad(const void* student_bf16, const void* teacher_bf16, const uint8_t* loss_mask,
                                  int64_t T, int64_t H, int32_t kind, float weight, const float* grad_loss_device,
                                  float denom_override, int32_t accumulate, void* workspace, size_t workspace_bytes,
                                  float* loss_out, float* loss_per_token, void* dstudent_bf16, void* cuda_stream);

/* The same record with one projection instead of two: the first sweep also stores the fp32 logits of the pass
 * (4096 tokens at a time) and the candidates are collected from them instead of being recomputed. Costs
 * 4096 x V x 4 bytes more workspace (2 GiB at V = 131072); same results, same limits, same errors. */
size_t kdkl_teacher_topk_stored_workspace_bytes(int64_t T, int64_t H, int64_t V, int32_t K);
int kdkl_teacher_topk_stored(const void* hidden_bf16, const void* weight_bf16, int64_t T, int64_t H, int64_t V,
                             int32_t K, float temperature, void* workspace, size_t workspace_bytes,
                             int32_t* topk_idx, float* topk_val, float* lse, void* cuda_stream);

/* Exercises the bounded wait every kernel of this library uses on its mbarriers: one thread waits on
 * a barrier that nothing completes, gives up after limit_ns (1 .. 1e9) and the kernel returns normally.
 * status: device int32[2], zeroed by the caller; afterwards {KDKL_ERR_TIMEOUT, 99}. The context stays
 * usable. (No counterpart in the paper: failure handling of this implementation.) */
int kdkl_wait_selftest(int32_t* status, int64_t limit_ns, void* cuda_stream);

/* Text of the last KDKL_ERR_CUDA on this thread. */
const char* kdkl_last_error(void);

/* Number of kernels the last forward / backward / host call on this thread enqueued. */
int64_t kdkl_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* KDKL_H_ */
