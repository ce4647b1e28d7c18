/*
 * deer.h -- C ABI of the DEER draft-verify hot path for NVIDIA B200 (sm_100a).
 *
 * One draft-verify cycle of the paper's inference routine (Section 3.2,
 * Algorithm 1) is: a block of k <= 32 draft tokens proposed for the prefix
 * x_{1:j}; the verifier's distributions p_AR(. | x_{1:j+i-1}), i = 1..k, from
 * one parallel pass; the acceptance rule (Eq. 5, Eq. 6); the accepted tokens
 * appended to the prefix.  This library holds the data-parallel parts of that
 * cycle as four calls -- deer_block_attn, deer_lmhead_select, deer_accept,
 * deer_kv_commit (with deer_kv_reserve as its counterpart) -- over a paged
 * bf16 KV cache that represents the prefix.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its comment says "host".  The
 *     caller owns all memory; the library allocates no device memory.
 *   - Every call returns an int status (DEER_OK = 0), validates its arguments
 *     on the host before launching, and is asynchronous on the CUDA stream
 *     passed last as `void*` (a cudaStream_t; NULL = the default stream).
 *   - Data-dependent failures (page pool exhausted, a page id out of range)
 *     are written by the kernels to the cache's device status word and read
 *     with deer_kv_status(); kernels never trap and never spin unboundedly.
 *   - Tensors are dense, row-major, last index fastest, 16-byte aligned.
 *     bf16 tensors are passed as `void*`.
 *   - Shapes: B sequences in the call, k block rows (1..32), Hq query heads,
 *     Hkv KV heads (Hq % Hkv == 0; query head h reads KV head h / (Hq/Hkv)),
 *     D head dim (64 or 128), page size 16 tokens, M = B*k rows, V vocabulary,
 *     hid hidden size (multiple of 64).
 */
#ifndef DEER_H_
#define DEER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DEER_OK               0
#define DEER_ERR_INVALID_ARG  1   /* null pointer, misaligned pointer, bad size              */
#define DEER_ERR_UNSUPPORTED  2   /* k > 32, head dim not 64/128, page size not 16, ...       */
#define DEER_ERR_NO_PAGES     3   /* device status: reserve found too few free pages          */
#define DEER_ERR_CUDA         4   /* a CUDA runtime call failed; see deer_last_error()        */
#define DEER_ERR_WORKSPACE    5   /* workspace smaller than the *_workspace_bytes() figure    */
#define DEER_ERR_BAD_PAGE     6   /* device status: a kernel met an unmapped/out-of-range page */
#define DEER_ERR_TIMEOUT      7   /* device status: a bounded wait inside a kernel ran out      */

#define DEER_MASK_CAUSAL 0   /* verifier: block row i sees block rows j <= i           */
#define DEER_MASK_BIDIR  1   /* drafter single-step fill: every block row sees all k   */

#define DEER_SEL_ARGMAX          0   /* ids only (temperature 0)                         */
#define DEER_SEL_ARGMAX_LOGPROB  1   /* ids + fp32 log-probability of the argmax (T = 1) */
#define DEER_SEL_SOFTMAX         2   /* ids + logsumexp(z/T) + draft-token logit (+ logits) */

#define DEER_ACC_GREEDY 0
#define DEER_ACC_SAMPLE 1
#define DEER_ACC_SAMPLE_PRESTATS 2 /* SAMPLE, the drafter statistics already in the workspace (deer_draft_stats) */
#define DEER_ACC_BONUS 4           /* or-ed into the mode: the k rows are k-1 drafts and one more row (see deer_accept) */
#define DEER_EMIT_PENDING 1        /* deer_emit flag: row 0 of the block was the token emitted last */

#define DEER_MAX_BLOCK 32
#define DEER_PAGE_SIZE 16

/* Text of the last host-side error of the calling thread (host pointer, never NULL). */
const char* deer_last_error(void);

/* ------------------------------------------------------------------------
 * Paged KV cache = the committed prefix x_{1:j} of each sequence
 * (Section 3.2, the step after Eq. 6; Algorithm 1's update of j).
 *
 * State, all caller-allocated device arrays described by deer_kv_desc:
 *   k_pool, v_pool  bf16 [num_pages][Hkv][16][D]
 *   page_table      i32  [max_seqs][max_pages]   physical page of logical page p, -1 if unmapped
 *   seq_len         i32  [max_seqs]              committed tokens n_s
 *   n_pages         i32  [max_seqs]              mapped logical pages (>= ceil(n_s/16))
 *   free_stack      i32  [num_pages]             free page ids in [0, *free_top); a pop takes the top
 *   free_top        i32  [1]
 *   status          i32  [1]                     0, or the first DEER_ERR_* a kernel recorded
 * Token t of sequence s lives at pool[page_table[s][t/16]][h][t%16][:].
 * The handle is a small host struct; destroying it frees nothing on the device.
 * ---------------------------------------------------------------------- */
typedef struct deer_kv deer_kv;

typedef struct deer_kv_desc {
    void*    k_pool;
    void*    v_pool;
    int32_t* page_table;
    int32_t* seq_len;
    int32_t* n_pages;
    int32_t* free_stack;
    int32_t* free_top;
    int32_t* status;
    int32_t  num_pages;
    int32_t  n_kv_heads;
    int32_t  head_dim;
    int32_t  page_size;
    int32_t  max_seqs;
    int32_t  max_pages;
} deer_kv_desc;

/* `desc` is a host pointer; its contents are copied. */
int deer_kv_create(deer_kv** kv, const deer_kv_desc* desc);
int deer_kv_destroy(deer_kv* kv);

/* Map pages so that each listed sequence can hold seq_len + k tokens:
 * sequences in the order of seq_ids, logical pages ascending, each page popped
 * from the top of the free stack.  If the free stack or max_pages is too small
 * nothing changes and the status word becomes DEER_ERR_NO_PAGES.
 * seq_ids: i32 [B], distinct.  B <= 1024. */
int deer_kv_reserve(deer_kv* kv, const int32_t* seq_ids, int B, int k, void* stream);

/* (4) Commit / roll back (Algorithm 1's update of j): seq_len[s] += keep[b]
 * with keep clamped to [0, k]; block rows written at positions >= the new length
 * are thereby dropped, and pages wholly beyond it return to the free stack --
 * sequences in order, logical pages descending.  `keep` is a device array
 * (e.g. deer_accept's accept_len), so no host round-trip is needed. */
int deer_kv_commit(deer_kv* kv, const int32_t* seq_ids, const int32_t* keep, int B, int k, void* stream);

/* (3) + (4) in one launch for greedy verification: deer_accept(DEER_ACC_GREEDY [| DEER_ACC_BONUS]) followed by
 * deer_kv_commit(keep = accept_len), same arguments, same results in accept_len / out_ids / n_out and in the cache
 * (Section 3.2's exact-match rule, Algorithm 1's update of j).  All arrays are device pointers; B <= 1024.
 * Errors: DEER_ERR_UNSUPPORTED for any other mode or size; the cache's status word as deer_kv_commit. */
int deer_accept_commit(deer_kv* kv, const int32_t* seq_ids, int mode, int B, int k, const int32_t* draft_ids,
                       const int32_t* target_ids, int32_t eos_id, int32_t* accept_len, int32_t* out_ids, int32_t* n_out,
                       void* stream);

/* Copy the status word to *code (host pointer) after synchronising `stream`,
 * and reset it to 0 on the device. */
int deer_kv_status(deer_kv* kv, int32_t* code, void* stream);

/* Self-test of the bounded waits (no counterpart in the paper): one thread block waits on a barrier that nothing
 * arrives on, with the same wait the tensor-core kernels use; the wait gives up after its limit (about a second of
 * SM clocks), the block raises DEER_ERR_TIMEOUT in the cache's status word and returns, and the context stays
 * usable.  Asynchronous on `stream`; read the outcome with deer_kv_status(). */
int deer_selftest_bounded_wait(deer_kv* kv, void* stream);

/* ------------------------------------------------------------------------
 * (1) Block attention (Section 3.2: the verifier scores all k block
 * positions in one pass, p_AR(. | x_{1:j+i-1}); the drafter fills the k masked
 * positions jointly from x_{1:j}).  For sequence b, head h, block row i:
 *     out = softmax(scale * q . K^T) V
 * over the keys {cache tokens 0..n_b-1} U {block rows j allowed by `mask`},
 * fp32 accumulation, bf16 output.
 *   q            bf16 [B][k][Hq][D]
 *   k_blk,v_blk  bf16 [B][k][Hkv][D]    keys/values of the block rows themselves
 *   out          bf16 [B][k][Hq][D]
 *   append       1: also write k_blk/v_blk into the cache at token positions
 *                n_b .. n_b+k-1 (pages must have been reserved); seq_len is
 *                NOT changed -- deer_kv_commit decides how many rows survive.
 *   max_seq_len  host-known upper bound on n_b over the batch; it only steers
 *                how the context is split over thread blocks and sizes the
 *                workspace.  A sequence longer than it sets DEER_ERR_INVALID_ARG
 *                in the status word and is skipped.
 *   workspace    >= deer_block_attn_workspace_bytes(...) bytes, 16-byte aligned;
 *                holds the split-context partial results.
 * ---------------------------------------------------------------------- */
size_t deer_block_attn_workspace_bytes(int B, int k, int Hq, int Hkv, int D, int max_seq_len);

int deer_block_attn(deer_kv* kv, const int32_t* seq_ids,
                    const void* q, const void* k_blk, const void* v_blk, void* out,
                    int B, int k, int Hq, int mask, int append, float scale, int max_seq_len,
                    void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * (2) LM head + selection: z = h w^T (bf16 x bf16 -> fp32), the verifier's
 * p_AR = softmax(z / T) of Eq. 5, reduced on the fly.
 *   h  bf16 [M][hid]      w  bf16 [V][hid]
 *   out_ids          i32 [M]  argmax_v z (lowest index among equal maxima)
 *   out_max_logprob  f32 [M]  max z - logsumexp(z)         (DEER_SEL_ARGMAX_LOGPROB)
 *   out_lse          f32 [M]  logsumexp(z / temperature)   (DEER_SEL_SOFTMAX)
 *   out_draft_logit  f32 [M]  z[draft_ids[m]]              (DEER_SEL_SOFTMAX, draft_ids != NULL)
 *   out_logits       f32 [M][V], optional in any mode (NULL = not stored)
 * Outputs not used by `mode` may be NULL.  temperature > 0 (ignored for ARGMAX).
 * hid must be a multiple of 64 and V at least 16 (else DEER_ERR_UNSUPPORTED).
 *   workspace  >= deer_lmhead_workspace_bytes(...) bytes, 16-byte aligned,
 *              contents arbitrary: per-row partial results of the thread blocks
 *              that split the vocabulary, merged inside the same kernel by the
 *              block that finishes last.  One call at a time per workspace.
 * Error behaviour on the device: every wait inside the kernel is bounded (about a
 * second); a thread block whose wait runs out gives up, and every row it worked on
 * gets out_ids[m] = -2 (no valid id is negative) with the other outputs of that
 * row undefined.  The call itself still returns DEER_OK: it is asynchronous.
 * ---------------------------------------------------------------------- */
size_t deer_lmhead_workspace_bytes(int M, int hid, int V);

int deer_lmhead_select(const void* h, const void* w, int M, int hid, int V,
                       int mode, float temperature, const int32_t* draft_ids,
                       int32_t* out_ids, float* out_max_logprob, float* out_lse,
                       float* out_draft_logit, float* out_logits,
                       void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * LM head + selection WITHOUT any caller-provided scratch.  (The paper has no
 * counterpart to this call; it exists for the library's users.)
 *
 * For callers that cannot allocate device memory where they call the library --
 * a serving loop whose memory pool is sealed after start-up, a plug-in that
 * receives only its input and output buffers, code that must stay out of the
 * CUDA allocator -- the split-vocabulary partial results live in a fixed
 * array inside the library image instead of a workspace.  Same arguments,
 * outputs and results as deer_lmhead_select, minus the workspace.
 *   - M must not exceed DEER_STATIC_MAX_ROWS (deer_lmhead_static_max_rows());
 *     larger M returns DEER_ERR_UNSUPPORTED and launches nothing.
 *   - The array (2*148*DEER_STATIC_MAX_ROWS*16 bytes, about 1.2 MB) is held by
 *     every GPU that loads the library until the process exits.
 *   - The call allocates and frees nothing, on the device or through any
 *     library routine.  The first call on each device looks up the array's
 *     device address (with that device current); make that first call outside
 *     any stream capture (inside one it returns DEER_ERR_UNSUPPORTED and does
 *     nothing).
 *   - All calls on one GPU share the array, which keeps the previous call's
 *     contents; each call overwrites every slot it later reads and leaves its
 *     arrival counters at zero, so no clearing is needed, but two calls that
 *     overlap on the GPU (different streams) race on it -- serialise them.
 * ---------------------------------------------------------------------- */
#define DEER_STATIC_MAX_ROWS 256

size_t deer_lmhead_static_max_rows(void);

int deer_lmhead_select_static(const void* h, const void* w, int M, int hid, int V,
                              int mode, float temperature, const int32_t* draft_ids,
                              int32_t* out_ids, float* out_max_logprob, float* out_lse,
                              float* out_draft_logit, float* out_logits, void* stream);

/* ------------------------------------------------------------------------
 * (3) Acceptance rule (Eq. 5, Eq. 6, Algorithm 1 inner loop; the first
 * rejection ends the block because later rows were conditioned on the
 * rejected draft).
 * GREEDY (temperature 0): accept_len = longest prefix with draft == target;
 *   the emitted tokens are the accepted drafts followed, if accept_len < k, by
 *   target_ids at the first mismatch.
 * SAMPLE: alpha_i = min(1, p(y_i)/q(y_i)), p = softmax(target_logits/T),
 *   q = softmax(draft_logits); accept iff u[b][i] <= alpha_i; at the first
 *   rejection one token is drawn from max(0, p - q) normalised, by inverse CDF
 *   in vocabulary order with r[b]; if that mass is zero, from p.  (p and q are
 *   taken as fp32 exponentials of logit - log-sum-exp, their differences summed
 *   in fp64: the draw equals an exact evaluation's whenever r * S stays 1e-4 * S
 *   away from the edges of the drawn token's interval of the cumulative sum S.)
 * No extra token is emitted when all k are accepted (Algorithm 1 as printed).
 * With DEER_ACC_BONUS or-ed into the mode the block's k rows are k-1 drafts
 * followed by one more row whose input was the last draft: column k-1 of
 * draft_ids, draft_logits and u is ignored, and when all k-1 drafts are accepted
 * one more token is taken from that row's p itself (GREEDY: target_ids[b][k-1];
 * SAMPLE: inverse CDF of p with r[b]), so every block emits accept_len + 1
 * tokens -- the parallel pass has that distribution anyway.  If eos_id >= 0
 * nothing is emitted after the first emitted eos_id.
 *   draft_ids           i32 [B][k]
 *   target_ids          i32 [B][k]        GREEDY
 *   target_logits       f32 [B][k][V]     SAMPLE (deer_lmhead_select's out_logits)
 *   target_lse          f32 [B][k]        SAMPLE logsumexp(target_logits / T)
 *   target_draft_logit  f32 [B][k]        SAMPLE target_logits[b][i][draft_ids[b][i]]
 *   draft_logits        f32 [B][k][V]     SAMPLE
 *   u f32 [B][k] in (0,1);  r f32 [B] in (0,1)
 *   accept_len i32 [B];  out_ids i32 [B][k] (-1 padded);  n_out i32 [B]
 * ---------------------------------------------------------------------- */
size_t deer_accept_workspace_bytes(int mode, int B, int k, int V);

/* The drafter's side of Eq. 5, q(y_i): log-sum-exp of draft_logits[b][i][:] and
 * the draft token's logit for every block row, one streaming pass over
 * draft_logits, left in `workspace` (deer_accept's SAMPLE workspace, same size).
 * q is known before the verifier has run, so this call may be issued on another
 * stream while deer_block_attn / deer_lmhead_select run; the caller orders it
 * before deer_accept(DEER_ACC_SAMPLE_PRESTATS, ..., same workspace), which then
 * skips that pass, and after the previous deer_accept on that workspace.
 * Errors: as deer_accept. */
int deer_draft_stats(int B, int k, int V, const int32_t* draft_ids, const float* draft_logits,
                     void* workspace, size_t workspace_bytes, void* stream);

int deer_accept(int mode, int B, int k, int V,
                const int32_t* draft_ids, const int32_t* target_ids,
                const float* target_logits, const float* target_lse, const float* target_draft_logit,
                float temperature, const float* draft_logits, const float* u, const float* r,
                int32_t eos_id, int32_t* accept_len, int32_t* out_ids, int32_t* n_out,
                void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Top-k / nucleus truncation of the verifier's distribution ahead of the
 * acceptance rule (the sampling setting of Table 1 is a temperature; these are
 * its usual companions).  For every row of target_logits, p = softmax(z / T):
 *   top_k > 0:  keep {v : p[v] >= the top_k-th largest value of p};
 *   top_p < 1:  of what is left, renormalised, the smallest upper level set
 *               {v : p[v] >= t} whose mass reaches top_p.
 * Both are level sets, so tokens of equal probability stay or go together and the
 * result is one threshold per row: tau[m], the smallest kept logit (token v is
 * kept iff z[v] >= tau[m]), and lse_trunc[m] = log sum_{kept} exp(z[v] / T), the
 * log-sum-exp that normalises the kept part.  deer_accept_truncated() then runs
 * Eq. 5 / Eq. 6 on that truncated distribution: a draft outside it is rejected,
 * the residual is max(0, p' - q) with p' the truncated, renormalised p.
 *   target_logits f32 [M][V];  target_lse f32 [M] = logsumexp(z / T) (deer_lmhead_select's out_lse)
 *   tau, lse_trunc f32 [M]     out
 * top_k <= 0 or >= V and top_p >= 1 switch the respective truncation off.
 * No workspace.  Errors: DEER_ERR_INVALID_ARG for null / misaligned pointers,
 * temperature <= 0 or top_p <= 0.
 * ---------------------------------------------------------------------- */
int deer_truncate(int M, int V, const float* target_logits, const float* target_lse, float temperature, int top_k,
                  float top_p, float* tau, float* lse_trunc, void* stream);

/* deer_accept on a truncated verifier distribution: target_tau f32 [B][k] (deer_truncate's tau) or NULL (= deer_accept),
 * and target_lse must then be deer_truncate's lse_trunc.  SAMPLE modes only use target_tau. */
int deer_accept_truncated(int mode, int B, int k, int V,
                          const int32_t* draft_ids, const int32_t* target_ids,
                          const float* target_logits, const float* target_lse, const float* target_draft_logit,
                          const float* target_tau, float temperature, const float* draft_logits, const float* u,
                          const float* r, int32_t eos_id, int32_t* accept_len, int32_t* out_ids, int32_t* n_out,
                          void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * (5) Book-keeping of one pass of Algorithm 1's outer loop (it runs until an
 * EOS is emitted: the tokens chosen in this block join the output, then j is
 * updated).  For every sequence that has not finished:
 * out_ids[b][0 .. n_out[b]) (deer_accept's output, already cut after an EOS) is
 * appended to tokens[b] as far as max_new allows; the sequence finishes when an
 * appended token equals eos_id (eos_id < 0 disables) or when it holds max_new
 * tokens; keep[b] = min(accept_len[b], tokens appended) is what
 * deer_kv_commit should keep.  A finished sequence appends nothing and gets
 * keep[b] = 0, so it may stay in the batch of later passes.
 * flags & DEER_EMIT_PENDING: row 0 of the block was the token emitted last (its
 * keys and values were not in the cache yet) and rows 1.. the drafts; one more
 * row is then kept, keep[b] = 1 + min(accept_len[b], tokens appended).
 *   accept_len, n_out  i32 [B];  out_ids  i32 [B][k]
 *   tokens    i32 [B][max_new]  output tokens so far (caller fills it with -1 before the first pass)
 *   n_tokens  i32 [B]           their number           (caller zeroes it before the first pass)
 *   finished  i32 [B]           0 / 1                  (caller zeroes it before the first pass)
 *   keep      i32 [B]           out
 *   appended  i32 [B] or NULL   out: tokens that joined tokens[b] in this pass (what the drafter's cache has to
 *                               take in, see deer_refresh_rows)
 * ---------------------------------------------------------------------- */
int deer_emit(int B, int k, const int32_t* accept_len, const int32_t* out_ids, const int32_t* n_out,
              int32_t eos_id, int32_t max_new, int32_t* tokens, int32_t* n_tokens, int32_t* finished,
              int32_t* keep, int32_t* appended, int flags, void* stream);

/* ------------------------------------------------------------------------
 * The drafter's block beyond the single-step fill (Section 4, "Generative
 * capabilities": a block completed over several denoising iterations; the
 * appendix on the DLLM KV cache: a drafter-side cache of the finished tokens).
 * The paper gives no formulas for either; these are the block-diffusion
 * decoding rules it points to, cut down to what attention and cache need.
 *
 * Row states (i32 [B][k], bidirectional mask only):
 *    1  masked   still a mask token: sees the prefix and every row that holds something
 *    0  decoded  a fixed token: sees the prefix and the decoded rows only, so that
 *                nothing computed for it depends on rows that may still change
 *   -1  absent   holds nothing: no key, no query (its output row is unspecified)
 * deer_block_attn_rows is deer_block_attn with such states (NULL = all rows
 * masked = deer_block_attn).  With append = 1 only the decoded rows' keys and
 * values are written, row i at token position n_b + i as always; the caller
 * commits as many leading rows as are decoded.
 *
 * deer_refill: one iteration's decision.  Every masked row whose most likely
 * token ids[b][i] has log-probability logprob[b][i] >= log_threshold becomes
 * decoded and tokens[b][i] = ids[b][i]; if a sequence has masked rows but none
 * qualifies, its most confident masked row does (the lowest row among equals).
 * left[b] (optional) = rows still masked.  log_threshold = -INFINITY decodes all
 * at once (the single-step draft of Section 3.2).
 *
 * deer_refresh_rows: row_state[b][i] = 0 for i < appended[b], else -1 -- the
 * states of the pass that brings the drafter's cache up to date after a verify
 * step: the tokens that joined the output see each other and the drafter's
 * prefix, their keys and values are appended, and deer_kv_commit(keep =
 * appended) on the drafter's cache keeps them.
 * ---------------------------------------------------------------------- */
int deer_block_attn_rows(deer_kv* kv, const int32_t* seq_ids,
                         const void* q, const void* k_blk, const void* v_blk, void* out, const int32_t* row_state,
                         int B, int k, int Hq, int mask, int append, float scale, int max_seq_len,
                         void* workspace, size_t workspace_bytes, void* stream);
int deer_refill(int B, int k, const int32_t* ids, const float* logprob, float log_threshold,
                int32_t* row_state, int32_t* tokens, int32_t* left, void* stream);
int deer_refresh_rows(int B, int k, const int32_t* appended, int32_t* row_state, void* stream);

/* ------------------------------------------------------------------------
 * (6) The rest of a verifier layer around the block attention.  The paper takes
 * its verifiers (the Qwen3 family) as given; these are that family's public
 * pre-norm decoder layer, at the M = B k rows of a draft block.  bf16 in and
 * out, fp32 arithmetic, all stream-ordered.
 *
 * deer_linear: y[m][n] = sum_c x[m][c] w[n][c] (+ residual[m][n]), the Q/K/V,
 *   output, gate/up and down projections.  x bf16 [M][K], w bf16 [N][K],
 *   residual bf16 [M][N] or NULL, y bf16 [M][N]; K a multiple of 64, N >= 16.
 *   The LM-head kernels without their selection: weight-streaming for small M.
 *   (As there: a thread block whose bounded wait runs out leaves its output
 *   tiles unwritten; the call has no status word of its own.)
 *   With a workspace of deer_linear_workspace_bytes (may be NULL / 0: slower for
 *   few output columns) the contraction is cut into ranges whose fp32 partial
 *   products are summed by a second kernel, so that every SM streams weights
 *   even when N is only a few thousand.
 * deer_rmsnorm: y = x / sqrt(mean(x^2) + eps) * gamma over each row of
 *   x bf16 [M][hid]; gamma bf16 [hid].
 * deer_qk_norm_rope: in place on q bf16 [B][k][Hq][D] and k_blk bf16
 *   [B][k][Hkv][D]: if q_gamma / k_gamma (bf16 [D]) are given, RMSNorm over each
 *   head's D values first; then the rotary embedding at position
 *   seq_len[seq_ids[b]] + i: dimension d < D/2 pairs with d + D/2, the pair
 *   turns by position * theta^(-2d/D).
 * deer_swiglu: y[m][c] = silu(gate_up[m][c]) * gate_up[m][I + c];
 *   gate_up bf16 [M][2 I], y bf16 [M][I].
 * ---------------------------------------------------------------------- */
size_t deer_linear_workspace_bytes(int M, int K, int N);
int deer_linear(const void* x, const void* w, const void* residual, void* y, int M, int K, int N,
                void* workspace, size_t workspace_bytes, void* stream);
int deer_rmsnorm(const void* x, const void* gamma, void* y, int M, int hid, float eps, void* stream);
int deer_qk_norm_rope(deer_kv* kv, const int32_t* seq_ids, void* q, void* k_blk, const void* q_gamma,
                      const void* k_gamma, int B, int k, int Hq, float eps, float theta, void* stream);
/* As deer_qk_norm_rope, fed by ONE fused projection: qkv bf16 [B k][(Hq + 2 Hkv) D] holds each row's query heads,
 * then its key heads, then its value heads; q and k_blk receive the transformed heads, v_blk a copy of the rest. */
int deer_qkv_split_norm_rope(deer_kv* kv, const int32_t* seq_ids, const void* qkv, void* q, void* k_blk, void* v_blk,
                             const void* q_gamma, const void* k_gamma, int B, int k, int Hq, float eps, float theta,
                             void* stream);
int deer_swiglu(const void* gate_up, void* y, int M, int I, void* stream);

/* A projection and the row-wise step that follows it in the layer, as one call each (fewer kernels: at the few rows of a
 * draft block the layer is bound by launches as much as by the weight stream).  Same arithmetic and the same bf16
 * roundings as the separate calls.
 * deer_linear_qkv_rope: the fused Q/K/V projection of x bf16 [B k][hid] by w_qkv bf16 [(Hq + 2 Hkv) D][hid], then
 *   deer_qkv_split_norm_rope on its result.
 * deer_linear_residual_norm: y = x w^T + residual (bf16 [M][N], residual may be NULL), and, if gamma != NULL,
 *   y_norm = RMSNorm(y) * gamma -- the output or down projection together with the normalisation that opens the
 *   next sub-layer.
 * deer_linear_swiglu: y bf16 [M][I] = silu(g) * u with (g, u) = the columns (2 c, 2 c + 1) of x w_pairs^T; w_pairs bf16
 *   [2 I][hid] holds channel c's gate row at 2 c and its up row at 2 c + 1 (a layout the caller prepares once).
 *   workspace  >= deer_layer_workspace_bytes(M, K, N) bytes (N = the projection's output columns), 16-byte aligned. */
size_t deer_layer_workspace_bytes(int M, int K, int N);
int deer_linear_qkv_rope(deer_kv* kv, const int32_t* seq_ids, const void* x, const void* w_qkv, void* q, void* k_blk, void* v_blk,
                         const void* q_gamma, const void* k_gamma, int B, int k, int Hq, int hid, float eps, float theta,
                         void* workspace, size_t workspace_bytes, void* stream);
int deer_linear_residual_norm(const void* x, const void* w, const void* residual, const void* gamma, void* y, void* y_norm,
                              int M, int K, int N, float eps, void* workspace, size_t workspace_bytes, void* stream);
int deer_linear_swiglu(const void* x, const void* w_pairs, void* y, int M, int K, int I, void* stream);

/* The routed mixture-of-experts MLP of a Qwen3-MoE-style layer (the paper's largest verifier, Qwen3-30B-A3B, has one
 * in every layer) at M = B k rows:
 *   probabilities = softmax(x w_router^T) over the E experts (fp32);  each row's top_k experts, lowest index among
 *   equals, their probabilities renormalised to sum 1;
 *   y[m] = residual[m] + sum_j weight[m][j] * down_e( silu(gate_e(x[m])) * up_e(x[m]) ),  e = expert[m][j].
 *   x bf16 [M][hid];  w_router bf16 [E][hid];  w_gate_up bf16 [E][2 I][hid] (an expert's I gate rows, then its I up
 *   rows);  w_down bf16 [E][hid][I];  residual bf16 [M][hid] or NULL;  y bf16 [M][hid].
 *   E <= 256, top_k <= min(32, E), hid and I multiples of 64.
 * The rows are regrouped by expert and both projections run as grouped GEMMs that stream each chosen expert's
 * weights once; gate, up (each rounded to bf16, as a dense layer would store them), the activations and the expert
 * outputs are bf16, sums fp32.
 * deer_moe_route is the first stage alone: experts i32 [M][top_k] in order of falling probability, weights f32
 * [M][top_k] (renormalise = 0: the softmax probabilities themselves); its workspace holds the M x E fp32 logits.
 *   workspace  >= deer_moe_workspace_bytes(...) bytes (deer_moe_route: M * E * 4), 16-byte aligned, contents arbitrary. */
size_t deer_moe_workspace_bytes(int M, int hid, int E, int I, int top_k);
int deer_moe_route(const void* x, const void* w_router, int M, int hid, int E, int top_k, int renormalise,
                   int32_t* experts, float* weights, void* workspace, size_t workspace_bytes, void* stream);
int deer_moe_mlp(const void* x, const void* w_router, const void* w_gate_up, const void* w_down, const void* residual,
                 void* y, int M, int hid, int E, int I, int top_k, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * One whole greedy verify step with HOST inputs and outputs (Algorithm 1, one
 * iteration of the while loop on the verifier side): copies the block's
 * q/k_blk/v_blk, hidden states and draft ids from host memory to the device
 * staging buffers in `dev`, runs reserve -> block_attn(causal, append) ->
 * lmhead_select(argmax) -> accept(greedy) -> commit(keep = accept_len), and
 * copies accept_len / out_ids / n_out back.  Model state (w, the KV cache)
 * stays on the device.  Returns after the stream has been synchronised.
 * On a stream other than the legacy default one, with page-locked host
 * buffers, the first call with a given set of arguments records the copies and
 * kernels into a CUDA graph and later calls with the same arguments replay it
 * (one launch instead of sixteen enqueues); the graph belongs to the library
 * (a few of them are kept, the least recently used one is replaced).  Every
 * pointer and size of `kv`'s descriptor, of `dev` and of the argument list is
 * part of that key, so swapping any buffer records a new graph.  Not to be
 * called on a stream that is being captured.
 * Buffers that follow one another in memory on both the host and the device
 * side -- q, k_blk, v_blk in that order; accept_len, out_ids, n_out in that
 * order -- are moved by one copy instead of three; in the recorded form the
 * last kernel writes the results into the page-locked host buffers itself.
 * ---------------------------------------------------------------------- */
typedef struct deer_step_dev {
    void* q; void* k_blk; void* v_blk; void* attn_out;     /* bf16 staging, shapes as in deer_block_attn */
    void* h;                                               /* bf16 [M][hid] */
    int32_t* seq_ids;                                      /* i32 [B], already filled */
    int32_t* draft_ids; int32_t* target_ids;               /* i32 [B][k] */
    int32_t* accept_len; int32_t* out_ids; int32_t* n_out;
    void* attn_ws; size_t attn_ws_bytes;
    void* lm_ws;   size_t lm_ws_bytes;
} deer_step_dev;

int deer_verify_step_host(deer_kv* kv, const deer_step_dev* dev /*host struct*/,
                          const void* w /*device bf16 [V][hid]*/,
                          const void* q_host, const void* k_blk_host, const void* v_blk_host,
                          const void* h_host, const int32_t* draft_ids_host,
                          int B, int k, int Hq, int hid, int V, float scale, int max_seq_len,
                          int32_t* accept_len_host, int32_t* out_ids_host, int32_t* n_out_host,
                          void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DEER_H_ */
