/*
 * aj_verify — the verify-and-judge step of AutoJudge speculative decoding on one B200 (sm_100a).
 *
 * One call verifies, for each of B sequences, a window of K draft tokens against the target
 * model and reports how many leading draft tokens are kept and which token the target
 * emits next.  Notation: M = B*(K+1) rows of hidden states; row 0 of a sequence encodes the
 * last accepted token, row i+1 encodes draft token i; F = d_draft + d judge features.
 *
 * What a call computes (the paper's Section 2, greedy verification, relaxed as in Section 3.3):
 *   logit[b,j,v] = sum_k h_target[b,j,k] * W_lm[k,v]      never written to memory
 *   y[b,j]       = argmax_v logit[b,j,v]                   lowest index on ties
 *   mismatch at i when draft_tok[b,i] != y[b,i]            (the set I(x) of Section 3.1)
 *   at a mismatch only, the classifier of Section 3.2 is evaluated on the hidden states that
 *   encode the mismatching draft token, draft and target model concatenated:
 *       p = sigmoid(judge_b + judge_w . [h_draft[b,i+1,:] ; h_target[b,i+1,:]])   = P(important)
 *   and the mismatch is forgiven iff p < tau (tau <= 0 never forgives, tau >= 1 always does);
 *   accept_len[b] = number of leading positions that match or are forgiven; the first
 *   unforgiven mismatch and everything after it are rejected (Section 2);
 *   next_tok[b]   = y[b, accept_len[b]]  (the bonus token y[b,K] when all K pass).
 *
 * Conventions.  Every function returns an aj_status and never throws, aborts or traps the GPU.
 * All tensors are caller-owned, contiguous, row-major.  "device" pointers are CUDA device
 * memory on the handle's device; "host" pointers are ordinary (preferably pinned) host memory.
 * Nothing the caller passes is retained after the enqueued work has run.  aj_verify and
 * aj_verify_host enqueue work on the given stream and do not synchronise it unless stated.
 */
#ifndef AJ_VERIFY_H
#define AJ_VERIFY_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct aj_handle_s *aj_handle;

typedef enum {
    AJ_OK = 0,
    AJ_ERR_INVALID_ARG = 1, /* NULL where required, size out of range, shape differs from the handle's */
    AJ_ERR_UNSUPPORTED = 2, /* a valid request this build has no kernel for (alignment, layout) */
    AJ_ERR_WORKSPACE = 3,   /* B or K exceeds what the handle was created for */
    AJ_ERR_CUDA = 4,        /* a CUDA runtime or driver call failed (no device, out of memory, ...) */
    AJ_ERR_TIMEOUT = 5,     /* a bounded wait inside a kernel ran out; outputs of that call are invalid */
    AJ_ERR_NOT_SM100 = 6    /* the device is not compute capability 10.x */
} aj_status;

typedef enum { AJ_BF16 = 0, AJ_F32 = 1 } aj_dtype; /* storage type of h_target, h_draft and W_lm */

typedef enum {
    AJ_W_VD = 0, /* W_lm stored row-major [V, d]: one contiguous row per vocabulary entry */
    AJ_W_DV = 1  /* W_lm stored row-major [d, V] */
} aj_w_layout;

enum {
    AJ_FLAG_TIME_KERNELS = 2u, /* record CUDA events around the projection kernel (see aj_last_gemm_ms) */
    AJ_FLAG_NO_EXTRA_ROW = 16u /* the caller does not encode the last draft token (Section 3.2, design choice 1,
                                  second way): h_target and h_draft are [B, K, ...], target_tok and top1_val are
                                  [B, K]; a mismatch at the last position is rejected without the classifier
                                  (judge_p there is NaN); when all K tokens pass, next_tok is -1 (there is no
                                  row to predict a further token from) */
};

/* Comparison switches: they select a slower kernel for the same result and exist for tests and
 * measurements.  Not part of the interface a caller should build on. */
enum {
    AJ_FLAG_FORCE_SIMT = 1u, /* the plain fp32-accumulate CUDA-core kernel for the projection */
    AJ_FLAG_ONE_SM = 8u      /* keep batches of more than 128 rows on the one-SM kernel instead of the
                                two-SM (CTA pair) kernel */
};

/*
 * Create a handle for fixed model dimensions on CUDA device `device`.
 *   max_B, max_K  largest batch and window a later call may use (1 <= K <= 1024)
 *   d, d_draft, V target hidden width, draft hidden width (0 = the judge sees target features
 *                 only, as in the paper's appendix "vLLM Inference Implementation Details"), vocabulary size
 *   dtype, layout storage of the hidden states and of W_lm
 * The handle owns a small device workspace: 8 bytes per row (max_B*(max_K+1)) for the per-row
 * packed (max, argmax) keys, a status word, and staging buffers for aj_verify_host.  This is the
 * only place memory is allocated.  AJ_BF16 needs d % 8 == 0 and d_draft % 8 == 0; the tensor-core
 * path needs AJ_BF16 and d % 64 == 0, and for AJ_W_DV also V % 8 == 0 (rows of [d, V] must be 16-byte
 * aligned); anything else runs on the CUDA-core kernel.
 * Errors: AJ_ERR_INVALID_ARG, AJ_ERR_UNSUPPORTED, AJ_ERR_CUDA, AJ_ERR_NOT_SM100.
 */
aj_status aj_create(aj_handle *out, int device, int max_B, int max_K, int d, int d_draft, int V,
                    aj_dtype dtype, aj_w_layout layout, unsigned flags);

/*
 * One verify-and-judge cycle (Sections 2 and 3.3), device buffers, asynchronous on `cuda_stream`.
 *   h_target   [B, K+1, d]        device, dtype of the handle, 16-byte aligned
 *   h_draft    [B, K+1, d_draft]  device, row 0 of each sequence is never read; NULL iff d_draft == 0
 *   W_lm       d x V              device, layout of the handle, 16-byte aligned
 *   draft_tok  [B, K] int32       device; ids outside [0,V) are data, they never match
 *   judge_w    [d_draft + d] f32  device, ordered [draft features ; target features]
 *   judge_b, tau                  classifier bias and decision threshold, by value
 *   B, K, d, V                    this call's batch and window; d and V must equal the handle's
 *   accept_len [B] int32 out      in [0, K]
 *   next_tok   [B] int32 out      in [0, V)
 *   target_tok [B, K+1] int32 out optional (NULL ok): y
 *   top1_val   [B, K+1] f32 out   optional: the winning logit of each row (fp32 accumulate)
 *   judge_p    [B, K] f32 out     optional: p at every mismatching position, NaN elsewhere
 *   cuda_stream                   a cudaStream_t (NULL = default stream)
 * Outputs are valid once the stream has reached the end of the enqueued work.  The return value
 * covers what the host can see; a kernel-side timeout shows up in aj_last_status.
 * Calls on one handle share its workspace: calls that overlap on the GPU race.
 * Errors: AJ_ERR_INVALID_ARG (nothing enqueued), AJ_ERR_WORKSPACE, AJ_ERR_UNSUPPORTED, AJ_ERR_CUDA.
 */
aj_status aj_verify(aj_handle h, const void *h_target, const void *h_draft, const void *W_lm,
                    const int32_t *draft_tok, const float *judge_w, float judge_b, float tau,
                    int B, int K, int d, int V,
                    int32_t *accept_len, int32_t *next_tok, int32_t *target_tok,
                    float *top1_val, float *judge_p, void *cuda_stream);

/*
 * Fold the target half of the classifier into the LM-head projection (the paper's Section 3.2,
 * "Classifier model & training": the paper remarks that a linear classifier can be computed together
 * with the LM head, at next to no cost).  judge_w . [h_draft ; h_target] splits into a draft half and a
 * target half, and the target half, w_target . h_target[row], has the shape of one more logit.  This call
 * appends w_target = judge_w[d_draft ..] to the vocabulary as three bf16 rows b0 + b1 + b2 that add up to
 * w_target to fp32 precision (each the bf16 rounding of what the earlier ones leave); later cycles on
 * this handle compute their dot products with every row of h_target in one extra vocabulary block of the
 * projection kernel (tensor cores, fp32 accumulation; the rows lie past V and never enter the argmax)
 * and the judge kernel then reads only the h_draft rows of the mismatching positions (nothing when
 * d_draft == 0).  Results agree with the unfused path within the tolerance stated for judge_p.
 *   judge_w  [d_draft + d] f32 DEVICE: read by a small kernel enqueued on cuda_stream; later calls of
 *            aj_verify and its variants on this handle must pass weights with the same target half
 *            (the draft half and judge_b are still taken from each call).  NULL switches back.
 * Only on the tensor-core path (AJ_BF16, d % 64 == 0): AJ_ERR_UNSUPPORTED otherwise.  Ignored while the
 * top-K rule is in force.  Errors: AJ_ERR_INVALID_ARG, AJ_ERR_UNSUPPORTED, AJ_ERR_CUDA.
 */
aj_status aj_fuse_judge(aj_handle h, const float *judge_w, void *cuda_stream);

/*
 * Switch the acceptance rule of a handle to the top-K rule of the paper's Section 4.1 (the lossy
 * baseline it compares with): a mismatching draft token is accepted iff it is among the top_k most
 * likely tokens of the target, i.e. iff fewer than top_k vocabulary entries have a larger logit
 * (among equal logits the lower index ranks first; a draft token outside the vocabulary is never
 * accepted).  The classifier is then not consulted: judge_w and h_draft may be NULL and judge_b, tau
 * are ignored; judge_p, if given, receives the draft token's rank (as a float, 0 = the target's own
 * token) at every mismatching position and NaN elsewhere; a rank below top_k is exact, a rejected
 * token's is some value from top_k up to its rank (the count stops once top_k entries outrank it).  A cycle then launches three kernels (the
 * draft tokens' own logits, the projection with the count fused into its epilogue, the scan).
 * top_k = 0 switches back to the classifier.  Not available on vocabulary-parallel handles or with
 * AJ_FLAG_NO_EXTRA_ROW (AJ_ERR_UNSUPPORTED).  Errors: AJ_ERR_INVALID_ARG.
 */
aj_status aj_set_top_k(aj_handle h, int top_k);

/*
 * Sampled verification (the paper's Appendix A, "Generalization to sampling"): the target's token of
 * every row is drawn from softmax(logit / temperature) instead of being the greedy argmax, by the
 * Gumbel-max trick with noise that is a deterministic function of the random state, so that a draw
 * can be reproduced: token = argmax_v (logit[v] + temperature * g[v]).  For row j of the call
 * (j = b * rows per sequence + position) and vocabulary entry v:
 *     x = word (j mod 4) of Philox4x32-10 with key (seed low word, seed high word) and counter
 *         (v, j div 4, step low word, step high word);
 *     u = ((x >> 9) + 0.5) * 2^-23;   g = -ln(-ln u)      (fp32 on the device).
 * The noise is added in the projection kernels' epilogues before the argmax; logits are still never
 * written.  Everything downstream (mismatch test, classifier, accepted prefix, next token) uses the
 * drawn tokens; top1_val receives the winning noisy score.  `step` is the cycle counter of the next
 * cycle enqueued on the handle and advances by one with every cycle, so that consecutive cycles
 * draw independent noise; set it again to replay a cycle.  The draw does not depend on the kernel
 * chosen, on tiling or on vocabulary sharding (the ranks of a vocabulary-parallel group must be
 * given the same temperature, seed and step; replicas that verify different sequences should be given
 * different seeds, since every handle numbers its rows from zero).  temperature = 0 switches back to greedy
 * verification.  Errors: AJ_ERR_INVALID_ARG (NULL handle, negative or non-finite temperature),
 * AJ_ERR_UNSUPPORTED (together with the top-K rule).
 */
aj_status aj_set_sampling(aj_handle h, float temperature, uint64_t seed, uint64_t step);

/*
 * The cycle for a tree draft (the paper's Section 3.3, "Generality": the method applies to tree-based
 * speculative decoding; its appendix integrates it with EAGLE-2).  The N draft tokens of a sequence are
 * the nodes of a tree in topological order: parent[b, n] is -1 for a child of the root (the last
 * accepted token) or the index, below n, of another node.  Row 0 of h_target / h_draft encodes the
 * root and row n + 1 encodes node n (the caller computed them under the tree's attention mask).  Node
 * n matches iff draft_tok[b, n] equals the target's token of its parent's row; a mismatching node
 * is scored by the classifier on row n + 1 exactly as a window position is.  A node is accepted iff
 * its parent is accepted (the root always is) and it matches or p < tau.  Outputs: accept_len[b] =
 * depth of the deepest accepted node (0 if none; among equally deep nodes the lowest index wins),
 * best_node[b] = that node (-1 = the root; optional, may be NULL; its ancestors are the accepted
 * path), next_tok[b] = the target's token of that node's row.  A node whose parent index is outside
 * [-1, n) is never accepted and never scored.  With parent[b, n] = n - 1 this is aj_verify.
 * All other arguments, their layouts, asynchrony and errors as aj_verify (N in place of K: N <= max_K;
 * draft_tok, parent and judge_p are [B, N], target_tok and top1_val [B, N + 1]); parent is a device
 * pointer.  Works with aj_set_sampling; not with aj_set_top_k or AJ_FLAG_NO_EXTRA_ROW
 * (AJ_ERR_UNSUPPORTED).
 */
aj_status aj_verify_tree(aj_handle h, const void *h_target, const void *h_draft, const void *W_lm,
                         const int32_t *draft_tok, const int32_t *parent, const float *judge_w, float judge_b,
                         float tau, int B, int N, int d, int V,
                         int32_t *accept_len, int32_t *next_tok, int32_t *best_node, int32_t *target_tok,
                         float *top1_val, float *judge_p, void *cuda_stream);

/*
 * Fit the classifier (the paper's Section 3.2 "Classifier model & training", Section 4.1 and its appendix
 * on classifier ablations: a logistic regression with L2 regularisation, fitted as scikit-learn does with
 * coefficient C, e.g. 1e-4 for the 8B / 70B pair).  The result is the minimiser of
 *     f(w, b) = 1/2 w.w + C * sum_i log(1 + exp(-s_i (x_i.w + b))),   s_i = +1 if labels[i] != 0 else -1
 * (intercept not regularised), found by L-BFGS with every evaluation of f and its gradient done in one
 * pass of a kernel over X.
 *   X       [n, F] DEVICE, row-major, dtype as given; row i is the concatenation [h_draft ; h_target] of a
 *           mined mismatch, the layout judge_w expects.  16-byte aligned, F * element size a multiple of 16.
 *   labels  [n] DEVICE bytes, non-zero = important.
 *   w_out   [F] DEVICE fp32, b_out HOST: the fitted judge_w and judge_b.
 *   iters_out (HOST, optional, 2 ints) receives {iterations, evaluations}; stats_out (HOST, optional, 2 floats)
 *           {the largest absolute component of the gradient of f at the result, the milliseconds the
 *           evaluations' loss + gradient kernel took in total (CUDA events)}.
 * Stops when that component is <= tol, after max_iter iterations, or when no step lowers f any more
 * (evaluations are fp32 per row, fp64 across rows).  Synchronous.  The first fit on a device allocates a
 * workspace ((SMs + 2) * F floats of device memory, 2 * F floats of pinned host memory) that later fits on
 * that device reuse (it grows if a later fit needs more); aj_lr_release frees it.  Fits in one process
 * take turns.  Errors: AJ_ERR_INVALID_ARG, AJ_ERR_UNSUPPORTED (alignment, or rows wider than 48 KB: 24 576
 * features in bf16, 12 288 in fp32), AJ_ERR_NOT_SM100, AJ_ERR_CUDA.
 */
aj_status aj_lr_fit(int device, const void *X, const uint8_t *labels, long long n, int F, aj_dtype dtype, float C,
                    int max_iter, float tol, float *w_out, float *b_out, int *iters_out, float *stats_out,
                    void *cuda_stream);

/* Free the workspace aj_lr_fit keeps on `device` (-1: on every device).  Errors: AJ_ERR_INVALID_ARG, AJ_ERR_CUDA. */
aj_status aj_lr_release(int device);

/*
 * The same cycle for a caller whose per-cycle tensors live in host memory: h_target, h_draft and
 * draft_tok are HOST pointers and are copied to the handle's staging buffers; accept_len and
 * next_tok (and target_tok, if not NULL) are HOST pointers and are copied back.  W_lm and judge_w
 * are model parameters and stay DEVICE pointers.  The call synchronises `cuda_stream` before it
 * returns, so the host outputs are valid on return.  draft_tok and the outputs are used in place,
 * without a copy, when they are pinned host memory (cudaHostAlloc / cudaHostRegister); pageable
 * buffers work too and are copied.  Pinned, 16-byte aligned hidden states of up to 1 MB per cycle are
 * fetched by a kernel (one launch more, and faster than two copy operations at that size); larger or
 * pageable ones go through the copy engines.
 */
aj_status aj_verify_host(aj_handle h, const void *h_target_host, const void *h_draft_host,
                         const void *W_lm, const int32_t *draft_tok_host, const float *judge_w,
                         float judge_b, float tau, int B, int K, int d, int V,
                         int32_t *accept_len_host, int32_t *next_tok_host, int32_t *target_tok_host,
                         void *cuda_stream);

/*
 * Device-side status of the calls made so far on this handle: AJ_OK, or AJ_ERR_TIMEOUT if a
 * bounded wait in a kernel gave up.  Synchronises the handle's device; reading clears the word.
 */
aj_status aj_last_status(aj_handle h);

/*
 * With AJ_FLAG_TIME_KERNELS: duration in milliseconds of the projection kernel (the fused
 * LM-head GEMM + argmax) of the most recent call, from CUDA events recorded on that call's stream
 * directly around the launch.  Waits for that kernel to finish.  AJ_ERR_INVALID_ARG without the flag.
 */
aj_status aj_last_gemm_ms(aj_handle h, float *ms);

/*
 * With AJ_FLAG_TIME_KERNELS: mean and minimum duration (milliseconds) of the projection kernel
 * over the calls made since the previous read-out (the most recent 512 at most), and how many
 * calls that was; then starts a new series.  Waits for those kernels to finish.  min_ms may be NULL.
 */
aj_status aj_gemm_ms_stats(aj_handle h, float *mean_ms, float *min_ms, int *count);

/* Number of kernels of this library that the most recent aj_verify / aj_verify_host call launched
 * (the projection kernel and the judge kernel; one more under the top-K rule). */
int aj_last_launch_count(aj_handle h);

/*
 * How the two-SM projection kernel cuts a batch of M = B*(K+1) rows against a vocabulary of V entries
 * (host arithmetic only, no device needed; for tests and diagnostics).  out receives
 *   [0] blocks of 256 vocabulary entries        [1] row tiles
 *   [2],[3] row tile i holds out[2] + (i < out[3]) units of 16 rows
 *   [4] rows of h_target each SM of a pair stages per 64-column block and accumulator
 *   [5] groups the row tiles are walked in (each group against the whole vocabulary, so that a
 *       group's rows of h_target stay in L2)    [6],[7] group g holds out[6] + (g < out[7]) row tiles
 *   [8] 1 if each tile uses two accumulators, each with its own issuing warp, that share the staged
 *       block of W_lm (a tile then holds up to 512 rows; chosen for every batch of more than 256 rows),
 *       else 0 (one tile of at most 256 rows on one accumulator, double-buffered)
 *   [9] depth of the shared-memory ring, in stages; a stage holds two 64-column blocks of every operand
 *       where three such stages fit (tiles of up to 320 rows, d / 64 even), else one
 * Errors: AJ_ERR_INVALID_ARG.
 */
aj_status aj_pair_schedule(int M, int d, int V, int32_t out[10]);

/* Name of the projection kernel configuration the most recent call used: "umma_vm_128x32" ... "umma_vm_128x256"
 * (one SM per tile: 128 vocabulary entries x up to that many rows), "umma_pair_256x256" (CTA pairs) or "simt". */
const char *aj_last_gemm_path(aj_handle h);

/*
 * The cycle of aj_verify for callers that cannot allocate device memory.  (The paper has no
 * counterpart to this entry point; it exists for integration.)
 *
 * aj_create calls cudaMalloc for its workspace.  A caller that gave all device memory to its own
 * pool at start-up, that runs under a per-allocation memory audit, or whose allocator is frozen by
 * the time it needs a cycle verified cannot use a handle.  This function takes no handle and calls
 * no cudaMalloc, cudaFree or any allocating routine: its only scratch memory, one 8-byte key per row
 * of hidden states plus a 256-byte block (a status word, and the two words through which the CTA pairs
 * of the two-SM kernel share out their tiles), is a fixed array inside the library's device image, so
 * every GPU that loads the library holds AJ_STATIC_MAX_ROWS * 8 + 256 bytes (about 256 KB) until exit.
 *
 * Arguments are those of aj_create and aj_verify together; the device is the CURRENT CUDA device;
 * all pointers are device pointers with the layouts aj_verify documents; optional outputs may be
 * NULL.  dev_status (optional, device, int32) receives 0, or AJ_ERR_TIMEOUT if a bounded wait in a
 * kernel ran out; read it after the stream has finished.  Without it a timeout goes unreported (there
 * is no handle to ask), so pass it wherever the result matters.
 * The cycle runs on the same kernels, chosen the same way, as aj_verify runs it on a plain handle: the
 * one-SM tensor-core kernel up to 128 rows, the two-SM kernel above (AJ_BF16, AJ_W_VD, d % 64 == 0), the
 * CUDA-core kernel for everything else (AJ_F32, AJ_W_DV, other widths).  The variants a handle can be
 * switched to (top-K rule, sampling, tree drafts, the folded classifier, vocabulary sharding) need a
 * handle's workspace and are not offered here.
 *   B * (K + 1) > AJ_STATIC_MAX_ROWS  ->  AJ_ERR_WORKSPACE, nothing enqueued.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress) and
 * prepares the kernels; make that first call outside any stream capture.  Later calls only enqueue.
 * All calls on a device share the one array, which keeps the previous call's contents (this call
 * clears the part it uses, in stream order): two calls whose GPU work overlaps, on different
 * streams or from different threads, race on it.  Serialise them.
 */
#define AJ_STATIC_MAX_ROWS 32768
aj_status aj_verify_static(const void *h_target, const void *h_draft, const void *W_lm,
                           const int32_t *draft_tok, const float *judge_w, float judge_b, float tau,
                           int B, int K, int d, int d_draft, int V, aj_dtype dtype, aj_w_layout layout,
                           int32_t *accept_len, int32_t *next_tok, int32_t *target_tok,
                           float *top1_val, float *judge_p, int32_t *dev_status, void *cuda_stream);

/*
 * ---------------------------------------------------------------------------------------------
 * Vocabulary-parallel form: the LM head split by vocabulary entries over up to 8 GPUs of one node,
 * the layout of the paper's tensor-parallel deployments (Section 4.3: the 70B target on 4 GPUs, the
 * 405B target on 8).  GPU r holds rows [v_begin, v_begin + v_count) of W_lm, projects the same
 * h_target against them, and the per-row (max, argmax) keys of all GPUs are merged by one 64-bit
 * max.  The projection kernel performs the exchange itself: its last CTA stores this GPU's keys into
 * a slot of EVERY GPU's exchange buffer (peer stores over NVLink) and then the cycle number into a
 * flag there; each GPU's judge kernel waits (at most 2 s, then AJ_ERR_TIMEOUT in aj_last_status)
 * for all flags of its own buffer and reduces the slots.  Every GPU computes the same accept_len and
 * next_tok.  One process per GPU; all ranks make the same sequence of calls with the same B and K.
 *
 * Exchange buffers are caller-owned device memory of aj_shard_exchange_bytes() bytes, 256-byte
 * aligned, one per GPU, each mapped into every process (aj_ipc_export / aj_ipc_import, or any other
 * peer mapping).  exchange[g] is rank g's buffer as addressable from THIS device; exchange[rank] is
 * this GPU's own.  aj_create_sharded zeroes the own buffer: put a barrier over all ranks between
 * creating the handles and the first cycle, and between the last cycle and freeing the buffers.
 */

/* Bytes of one GPU's exchange buffer; 0 if an argument is out of range (world in 1..8). */
size_t aj_shard_exchange_bytes(int max_B, int max_K, int world);

/*
 * An exchange buffer on the CURRENT device, as its own cudaMalloc allocation (so that aj_ipc_export
 * describes exactly this buffer), zero-filled; and its release.  A caller may instead pass any
 * 256-byte aligned device memory of aj_shard_exchange_bytes() bytes that its peers can address.
 * Errors: AJ_ERR_INVALID_ARG, AJ_ERR_CUDA.
 */
aj_status aj_shard_exchange_alloc(int max_B, int max_K, int world, void **device_ptr_out);
aj_status aj_shard_exchange_free(void *device_ptr);

/* The contiguous vocabulary range of rank `rank` among `world` GPUs: whole blocks of 256 entries,
 * spread evenly.  Errors: AJ_ERR_INVALID_ARG (also when V has fewer than `world` blocks). */
aj_status aj_shard_range(int V, int world, int rank, int *v_begin, int *v_count);

/*
 * aj_create for one GPU of a vocabulary-parallel group.  V is the WHOLE vocabulary (token ids in
 * the outputs are global); this GPU's W_lm argument in later calls is its shard, v_count rows
 * (layout AJ_W_VD: [v_count, d]; AJ_W_DV: [d, v_count]).
 * Errors: as aj_create, and AJ_ERR_INVALID_ARG for a bad rank, range or buffer.
 */
aj_status aj_create_sharded(aj_handle *out, int device, int max_B, int max_K, int d, int d_draft, int V,
                            aj_dtype dtype, aj_w_layout layout, unsigned flags,
                            int rank, int world, int v_begin, int v_count, void *const *exchange);

/*
 * On a sharded handle aj_verify and aj_verify_host run a whole cycle (W_lm = this GPU's shard).
 * The two halves can also be enqueued separately: aj_shard_project enqueues the projection of the
 * shard and the exchange; aj_shard_finish enqueues the wait for all GPUs' keys, the judge and the
 * prefix scan.  Arguments as in aj_verify.  Every aj_shard_project must be followed by its
 * aj_shard_finish before the next cycle.  Errors: as aj_verify.
 */
aj_status aj_shard_project(aj_handle h, const void *h_target, const void *W_shard, int B, int K, void *cuda_stream);
aj_status aj_shard_finish(aj_handle h, const void *h_target, const void *h_draft, const int32_t *draft_tok,
                          const float *judge_w, float judge_b, float tau, int B, int K,
                          int32_t *accept_len, int32_t *next_tok, int32_t *target_tok,
                          float *top1_val, float *judge_p, void *cuda_stream);

/*
 * Sharing an exchange buffer between the processes of one node (thin wrappers over CUDA IPC, so that
 * a caller needs no CUDA binding of its own): export gives 64 opaque bytes for a cudaMalloc'ed
 * device pointer; import, in another process with its own device current, maps that memory and
 * enables peer access; close unmaps it.  Errors: AJ_ERR_INVALID_ARG, AJ_ERR_CUDA.
 */
aj_status aj_ipc_export(const void *device_ptr, unsigned char handle_out[64]);
aj_status aj_ipc_import(const unsigned char handle_in[64], void **device_ptr_out);
aj_status aj_ipc_close(void *device_ptr);

/* Free the handle and its workspace.  The caller must have synchronised all work using it. */
aj_status aj_destroy(aj_handle h);

const char *aj_status_string(aj_status s);
const char *aj_version(void);

#ifdef __cplusplus
}
#endif
#endif /* AJ_VERIFY_H */
