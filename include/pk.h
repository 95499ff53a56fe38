/*
 * pk.h -- C ABI of the packed-attention library for NVIDIA B200 (sm_100a).
 *
 * The library evaluates causal self-attention over a PACKED token stream: several
 * examples are concatenated into one sequence of T tokens, `position_ids` restart at
 * every example (Sec. 3 "Packing with Position IDs", Sec. 3.1), and every token
 * attends only to earlier tokens of its own example (Table 1, "Correct
 * Cross-Attention").  Example boundaries are recovered on the device from the
 * position ids (paragraph after Table 1: "compute cu_seq_len from position_ids").
 *
 * Conventions that hold for every call
 *   - All data pointers are DEVICE pointers unless the comment says "host".
 *   - Tensors are contiguous, row-major: q/out/dout/dq are [T, Hq, D]; k/v/dk/dv are
 *     [T, Hkv, D]; lse is [Hq, T] fp32.  Tensor pointers must be 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Everything is enqueued on it; no call synchronises except pk_status_read.
 *   - The caller owns every buffer.  The library allocates no device memory.
 *   - Return value: PK_OK or one of the host-detected PK_ERR_* codes.  Problems only
 *     the device can see (negative position ids, a pipeline wait that ran out) are
 *     recorded in the workspace's status word; the kernels then stop early and leave
 *     the outputs untouched.  Read it with pk_status_read.
 *   - Supported shapes: D a multiple of 16 up to 128; Hq % Hkv == 0; 0 <= T; T*Hq*D' < 2^31
 *     with D' = 64 for D <= 64, else 128.  The kernels are built for D = 64 and D = 128; any
 *     other D runs on zero-padded copies of the tensors kept in the workspace (which
 *     pk_workspace_bytes sizes for them): one extra streaming pass over every tensor each way
 *     and contractions at the padded size, same results.
 *   - Query head h reads kv head h / (Hq / Hkv).
 *   - Values of OTHER examples must be finite: a masked probability is exactly 0, but
 *     0 * Inf is NaN inside a tensor-core contraction.
 */
#ifndef PK_H_
#define PK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- return / status codes ------------------------------------------------------- */
#define PK_OK               0
#define PK_ERR_INVALID_ARG  1   /* null pointer, negative size, misaligned pointer      */
#define PK_ERR_UNSUPPORTED  2   /* head_dim / head counts / dtype outside the supported set */
#define PK_ERR_WORKSPACE    3   /* workspace smaller than pk_workspace_bytes            */
#define PK_ERR_CUDA         4   /* a CUDA runtime/driver call or launch failed          */
#define PK_ERR_BAD_POSIDS   5   /* device: a position id is negative (detail = index)   */
#define PK_ERR_TIMEOUT      6   /* device: a bounded pipeline wait ran out (detail = which) */
#define PK_ERR_NO_PLAN      7   /* device: reuse_plan=1 but the workspace holds no plan for this T */

/* ---- element types of outputs ---------------------------------------------------- */
#define PK_BF16 0
#define PK_F32  1

/* ---- workspace sections (pk_workspace_section) ----------------------------------- */
#define PK_WS_HEADER     0   /* int32[32]: see PK_HDR_* indices                        */
#define PK_WS_FWD_ITEMS  1   /* int32[T][4]  (q_start, q_len, kv_start, kv_len)        */
#define PK_WS_BWD_ITEMS  2   /* int32[T][4]  (kv_start, kv_len, q_start, q_len)        */
#define PK_WS_FWD_ORDER  3   /* int32[T]     item indices, longest example first       */
#define PK_WS_BWD_ORDER  4   /* int32[T]                                                */
#define PK_WS_DELTA      5   /* fp32 [Hq][T] row sums of dO*O                           */
#define PK_WS_DQ_ACC     6   /* fp32 [T+128][Hq][D] accumulator of dQ                   */
#define PK_WS_ROPE_TABLE 7   /* fp32 [T][D/2][2] (cos, sin) of pos * theta^(-2i/D)      */
#define PK_WS_NUM_SECTIONS 8

/* indices into the int32 header */
#define PK_HDR_STATUS      0
#define PK_HDR_DETAIL      1
#define PK_HDR_N_EXAMPLES  2
#define PK_HDR_MAX_SEQLEN  3
#define PK_HDR_N_ITEMS     4   /* forward and backward lists have the same length      */
#define PK_HDR_PLAN_T      5   /* T the plan was built for, -1 if none                  */

/*
 * Tile shape used by the work lists (rows of a query block, rows of a key block).
 * Not in the paper: the lists are how "tiles outside an example's causal block are
 * never scheduled" is made checkable.  Host pointers.  Always returns PK_OK.
 */
int pk_tile_shape(int32_t* bm, int32_t* bn);

/*
 * Bytes of workspace the other calls need for a stream of T tokens (upper bound over
 * every example layout).  Returns 0 for unsupported arguments.
 */
size_t pk_workspace_bytes(int32_t T, int32_t Hq, int32_t Hkv, int32_t D);

/*
 * Byte offset and size of one section of the workspace (PK_WS_*), so that a caller or
 * a test can look at the plan.  Host pointers.  PK_ERR_INVALID_ARG for a bad section.
 */
int pk_workspace_section(int32_t which, int32_t T, int32_t Hq, int32_t Hkv, int32_t D,
                         size_t* offset, size_t* bytes);

/*
 * Boundary recovery and planning (paragraph after Table 1; Sec. 3.1 for the form of
 * the ids).  Token t starts an example iff t == 0 or position_ids[t] <= position_ids[t-1].
 *   position_ids  int32 [T]
 *   cu_seqlens    int32 [T+1] out: the E start offsets, then T, then T in every
 *                 remaining entry
 *   n_examples    int32 [1] out (device): E
 *   max_seqlen    int32 [1] out (device): longest example
 *   workspace     >= pk_workspace_bytes(T, Hq, Hkv, D) bytes, 256-byte aligned.  Receives the
 *                 plan: forward items (a block of <= bm query rows of one example and
 *                 the key range [example start, last row] it may see), backward items
 *                 (a block of <= bn key rows and the query range up to the example end
 *                 that may see it), both in ascending (example, block) order, plus the
 *                 schedule order of the items: stable sort by descending tile count of the
 *                 item's example (long examples first, an example's items adjacent).
 * T == 0 is valid: cu_seqlens = [0], E = 0.  No host round trip; one kernel launch.
 */
int pk_seqlens_from_posids(const int32_t* position_ids, int32_t T,
                           int32_t* cu_seqlens, int32_t* n_examples, int32_t* max_seqlen,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Rotary embedding indexed by position_ids, in place (unfused form of what the
 * attention calls do while loading Q/K tiles).  The paper only requires that models
 * "expose position IDs" (end of Sec. 3.5); the rotation is the usual one:
 * pairs (i, i + D/2), angle position_ids[t] * theta^(-2i/D); inverse != 0 rotates by
 * the negative angle.   x: bf16 [T, H, D].  D even, <= 256.
 */
int pk_rope_apply(void* x, const int32_t* position_ids, int32_t T, int32_t H, int32_t D,
                  float theta, int32_t inverse, void* stream);

/*
 * Forward (Sec. 3, Table 1 "Correct Cross-Attention"): for every query head h and
 * token i of example e,  S_ij = softmax_scale * <q'_i, k'_j> for s_e <= j <= i,
 * lse[h][i] = log sum_j exp S_ij (natural log),  out[i][h] = sum_j exp(S_ij - lse) v_j.
 *   q, k, v       bf16
 *   rope_theta    > 0: q and k are rotated by position_ids while their tiles are loaded
 *                 (q', k'); <= 0: q and k are used as given
 *   window        0: every row sees all keys of its example up to itself.  > 0: only its `window`
 *                 most recent keys, its own position included (sliding-window attention of
 *                 the Mistral family; the paper lists the model, the definition is that
 *                 model's).  Key tiles that no row of a query block can see are skipped.
 *                 Not available with pk_set_rope_mode(PK_ROPE_IN_TILE) and rope_theta > 0
 *                 (PK_ERR_UNSUPPORTED); pk_attn_bwd must be given the forward's value.
 *   out           [T, Hq, D], element type out_dtype (PK_BF16 or PK_F32)
 *   lse           fp32 [Hq, T]
 *   reuse_plan    bit mask.  0: run the planning step of pk_seqlens_from_posids first (same
 *                 stream); PK_REUSE_PLAN: use the plan already in `workspace` (must be for
 *                 these position_ids).  pk_attn_bwd also takes PK_REUSE_ROTATED: with
 *                 rope_theta > 0 the forward leaves rotated copies of q and k in the workspace
 *                 (default RoPE mode); the flag says that they are
 *                 still there (same q, k, position_ids, rope_theta; workspace untouched since
 *                 the forward), so the backward does not make them again.  For a padded head
 *                 size the flag covers the forward's padded copies of q, k and v in the same
 *                 way (with or without RoPE).
 */
#define PK_REUSE_PLAN     1
#define PK_REUSE_ROTATED  2
int pk_attn_fwd(const void* q, const void* k, const void* v, const int32_t* position_ids,
                int32_t T, int32_t Hq, int32_t Hkv, int32_t D,
                float softmax_scale, float rope_theta, int32_t window,
                void* out, int32_t out_dtype, float* lse,
                int32_t reuse_plan, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward of pk_attn_fwd: given dout = dL/dout, computes dq, dk, dv.  A row-sum
 * pre-pass forms delta = sum_d dout*out; the main kernel recomputes the probabilities
 * from lse, dV = P^T dO, dP = dO V^T, dS = P o (dP - delta), dQ = scale dS K',
 * dK = scale dS^T Q'; dK and dV are summed over the Hq/Hkv query heads of a kv head.
 * With rope_theta > 0 the gradients are with respect to the un-rotated q and k.
 *   out, out_dtype   the forward's output as it was written
 *   dq [T,Hq,D], dk, dv [T,Hkv,D]   element type grad_dtype (PK_BF16 or PK_F32)
 * The backward runs as two kernels, one key-block stationary for dK/dV and one query-block
 * stationary for dQ; every gradient is accumulated in a fixed order and is bitwise
 * reproducible.  With rope_theta > 0 they work on rotated copies of q and k (made by a
 * streaming pass, or left by the forward: PK_REUSE_ROTATED) and rotate dQ / dK back as they
 * write them.  Only with pk_set_rope_mode(PK_ROPE_IN_TILE) one kernel produces all three and
 * dQ goes through fp32 reductions in the workspace (order not fixed) followed by a scale /
 * un-rotate / cast pass.
 */
int pk_attn_bwd(const void* dout, const void* q, const void* k, const void* v,
                const void* out, int32_t out_dtype, const float* lse,
                const int32_t* position_ids,
                int32_t T, int32_t Hq, int32_t Hkv, int32_t D,
                float softmax_scale, float rope_theta, int32_t window,
                void* dq, void* dk, void* dv, int32_t grad_dtype,
                int32_t reuse_plan, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Copies the workspace's status word to the host and waits for `stream` (the only call
 * that synchronises).  code/detail are host pointers: PK_OK, or the first device-side
 * error recorded since the last planning step.
 */
int pk_status_read(const void* workspace, void* stream, int32_t* code, int32_t* detail);

/*
 * How the attention calls apply RoPE when rope_theta > 0 (process-wide; the paper is silent on
 * RoPE, both modes compute the same function):
 *   PK_ROPE_ROTATED_COPIES (default)  one pass writes rotated fp16 copies of q and k into the
 *       workspace (it reuses the PK_WS_DQ_ACC section), then the warp-specialised kernels run
 *       on them and rotate dQ/dK back in their epilogues.  A K tile is visited by every query
 *       tile of every head of its group, so rotating once costs one HBM pass instead of one
 *       rotation per visit.  Every supported shape.
 *   PK_ROPE_IN_TILE  the Q/K tiles are rotated in shared memory right after their TMA load
 *       (D = 64 and 128 only: padded head sizes always take the rotated copies; no sliding
 *       window).
 */
#define PK_ROPE_ROTATED_COPIES 0
#define PK_ROPE_IN_TILE        1
int pk_set_rope_mode(int32_t mode);

/*
 * pk_seqlens_from_posids for callers that cannot give the library a workspace and for whom
 * a device allocation is not an option (the paper has no counterpart; it is the same
 * boundary recovery as pk_seqlens_from_posids with the same outputs).  Typical callers: a
 * collation or data-loading thread that wants cu_seqlens for the next batch while the
 * training framework's caching allocator already holds nearly all device memory, so that a
 * cudaMalloc from a side library may fail; and latency-sensitive loops, because
 * cudaMalloc/cudaFree synchronise the whole device.  This call allocates nothing and frees
 * nothing: its scratch is a fixed array inside the library, PK_NOALLOC_MAX_TOKENS tokens
 * large (about 1.6 MB, resident on every GPU that loads the library until the process ends).
 *   - T > PK_NOALLOC_MAX_TOKENS returns PK_ERR_TOO_LARGE and launches nothing.
 *   - The first call on each device looks up the array's device address (one-time set-up,
 *     with that device current); make that first call before any stream capture begins.
 *   - All calls on a device share the one array: two calls whose kernels can overlap on the
 *     GPU (different streams without an ordering between them) race.  Order them.
 *   - Only cu_seqlens, n_examples and max_seqlen are delivered; the attention calls still
 *     take a caller workspace and plan for themselves.
 * Arguments as for pk_seqlens_from_posids.
 */
#define PK_NOALLOC_MAX_TOKENS 32768
#define PK_ERR_TOO_LARGE      8   /* size beyond a fixed built-in capacity */
int pk_seqlens_from_posids_noalloc(const int32_t* position_ids, int32_t T,
                                   int32_t* cu_seqlens, int32_t* n_examples,
                                   int32_t* max_seqlen, void* stream);

/* ---- steps around the attention path (the scope's "next" rows) -------------------------- */

/*
 * Padding-free collator (Sec. 3.4 "PaddingFreeCollator", worked example in Sec. 3.5), on the
 * device: the examples are already concatenated in input_ids; from their lengths it writes
 *   cu_seqlens   int32 [E+1]  prefix sums of the lengths (cu_seqlens[0] = 0)
 *   position_ids int32 [T]    0 .. L_e-1 for every example
 *   labels       int32 [T]    input_ids with the first entry of every example replaced by
 *                             ignore_index (the paper uses -100); may be NULL
 * All pointers are device pointers.  Requires sum(lengths) == T and E >= 1 when T > 0.
 */
int pk_collate_padding_free(const int32_t* input_ids, const int32_t* lengths, int32_t E, int32_t T,
                            int32_t* position_ids, int32_t* labels, int32_t* cu_seqlens,
                            int32_t ignore_index, void* stream);

/*
 * Fixed-length packing with position ids (Sec. 3.3 and Table 1: the packing variant that uses
 * position ids but still breaks examples): as pk_collate_padding_free, and in addition the stream
 * is cut into packs of msl tokens (pack k = tokens [k*msl, (k+1)*msl); the last one may be
 * short).  The paper does not describe the ids of the tail of a broken example; here a pack is a
 * sequence of its own, so the fragment that opens a pack is a new example: its position ids
 * restart at 0 and its first label becomes ignore_index.  cu_seqlens still receives the prefix
 * sums of the given lengths ([E+1]); the boundaries the attention calls use are the ones they
 * recover from position_ids (example starts and pack starts).  msl <= 0 is PK_ERR_INVALID_ARG.
 */
int pk_collate_fixed_length(const int32_t* input_ids, const int32_t* lengths, int32_t E, int32_t T,
                            int32_t msl, int32_t* position_ids, int32_t* labels,
                            int32_t* cu_seqlens, int32_t ignore_index, void* stream);

/*
 * Sample selection (Sec. 3.3), on the HOST (all pointers are host pointers): bin_of[i] receives
 * the pack of example i, *n_bins the number of packs.  Every length must be in [1, capacity].
 *   first_fit_decreasing  Multipack-style: examples from long to short (ties in the given
 *                         order), each into the first pack with room
 *   next_fit              first-come-first-served in the given order (sort_descending = 0, the
 *                         random-order baseline) or from long to short (sort_descending = 1,
 *                         the sorted baseline); a new pack starts when the next example does
 *                         not fit.  Examples are never broken.
 */
int pk_pack_first_fit_decreasing(const int32_t* lengths, int32_t n, int32_t capacity,
                                 int32_t* bin_of, int32_t* n_bins);
int pk_pack_next_fit(const int32_t* lengths, int32_t n, int32_t capacity, int32_t sort_descending,
                     int32_t* bin_of, int32_t* n_bins);

/*
 * Between a padded batch and the packed stream (for comparing the two layouts on whole models).
 * The padded layout is the one the paper starts from (Sec. 3: examples extended to the longest one
 * with padding appended on the right), the packed one the concatenation of Sec. 3.4.  Rows are
 * opaque `row_bytes` bytes each (a token id, a hidden vector, ...); device pointers throughout.
 *   pk_pack_rows     packed[cu[b] + i] = padded[b][i]  for i < cu[b+1] - cu[b]
 *   pk_unpack_rows   padded[b][i] = packed[cu[b] + i] for those i, zero bytes in the padding rows
 * padded is [B][l_max][row_bytes], packed [T][row_bytes], cu_seqlens int32 [B+1] with
 * cu_seqlens[B] = T and every length <= l_max (not checked).  16-byte copies when row_bytes and
 * both pointers allow it, else 4-byte or single bytes.
 */
int pk_pack_rows(const void* padded, const int32_t* cu_seqlens, int32_t B, int32_t l_max, int32_t T,
                 int64_t row_bytes, void* packed, void* stream);
int pk_unpack_rows(const void* packed, const int32_t* cu_seqlens, int32_t B, int32_t l_max, int32_t T,
                   int64_t row_bytes, void* padded, void* stream);

/*
 * Loss of the packed stream (the step right after the model).  The collator's labels carry -100
 * in the first position of every example (Sec. 3.4, worked example in Sec. 3.5); a causal
 * language model scores row t against the label of row t + 1, so with those labels no example
 * is asked to predict the start of the next one:
 *   target[t] = labels[t + 1] for t < T - 1, none for the last row; rows whose target equals
 *   ignore_index (or is not a vocabulary index) do not count
 *   loss_t = log(sum_v exp(logits[t][v])) - logits[t][target[t]],  loss = sum_t loss_t / n_valid
 * pk_packed_loss_fwd   logits [T][row_stride] (PK_BF16 or PK_F32, row_stride >= V elements; rows
 *                      are read with 16-byte loads when V, row_stride and the base allow it),
 *                      labels int32 [T].  Writes token_loss float [T] (0 for rows without a
 *                      target), lse float [T] (natural-log logsumexp, 0 for those rows),
 *                      result float [2] = {mean, sum}, n_valid int32 [1].  The sum runs in a
 *                      fixed order: the scalars are bitwise reproducible.  T == 0 gives 0, 0, 0.
 * pk_packed_loss_bwd   dlogits[t][v] = (exp(logits[t][v] - lse[t]) - [v == target[t]]) * grad_out
 *                      / n_valid for rows with a target, 0 for the others; same dtype and stride
 *                      as logits (columns >= V of a padded row are left untouched).  lse and
 *                      n_valid are the forward's outputs (device pointers: no host round trip).
 * All pointers are device pointers; the calls allocate nothing.
 */
int pk_packed_loss_fwd(const void* logits, int32_t logits_dtype, const int32_t* labels, int32_t T,
                       int32_t V, int64_t row_stride, int32_t ignore_index, float* token_loss,
                       float* lse, float* result, int32_t* n_valid, void* stream);
int pk_packed_loss_bwd(const void* logits, int32_t logits_dtype, const int32_t* labels,
                       const float* lse, const int32_t* n_valid, float grad_out, int32_t T, int32_t V,
                       int64_t row_stride, int32_t ignore_index, void* dlogits, void* stream);

/*
 * Self-test of the bounded waits (no counterpart in the paper): one small kernel waits on a
 * barrier that nothing will ever signal, for at most `budget_cycles` SM clocks (1 .. 2e9), then
 * records PK_ERR_TIMEOUT (detail 99) in the status word of `workspace` (>= 128 bytes, its header
 * must have been initialised by a planning call) and returns normally -- the same path a stuck
 * pipeline takes inside the attention kernels.  The context stays usable.
 */
int pk_selftest_bounded_wait(void* workspace, int64_t budget_cycles, void* stream);

/*
 * Measurement aid (no counterpart in the paper): asks the library to record the CUDA
 * events `start` and `stop` (cudaEvent_t passed as void*, owned by the caller) on the
 * call's stream immediately before and after every later launch of kernel `which`
 * (PK_KERNEL_*), so that a benchmark can time one kernel inside a multi-kernel call.
 * Pass NULL for both to stop recording.  Process-wide and not thread-safe.
 */
#define PK_KERNEL_PLAN      0
#define PK_KERNEL_FWD       1
#define PK_KERNEL_DELTA     2
#define PK_KERNEL_BWD       3   /* dK/dV kernel (the whole backward when RoPE is fused) */
#define PK_KERNEL_DQ_FINISH 4
#define PK_KERNEL_BWD_DQ    5   /* dQ kernel */
#define PK_KERNEL_LOSS_FWD  6   /* row pass of pk_packed_loss_fwd */
#define PK_KERNEL_LOSS_BWD  7
#define PK_NUM_KERNELS      8
int pk_set_timing_events(int32_t which, void* start, void* stop);

#ifdef __cplusplus
}
#endif
#endif /* PK_H_ */
