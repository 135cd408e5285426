/*
 * vscan.h - C ABI of the VScan visual-token reduction library for NVIDIA B200 (sm_100a).
 *
 * The library implements the two reduction points of VScan:
 *   Stage 1 (Sec. 4.1), at the vision-encoder output, per encoder instance (image or crop):
 *     vscan_score (ROW mode)        head mean of the [CLS] attention rows          (Eq. 1-2)
 *     vscan_select_global_local     per-window top-k + global top-k, union         (Eq. 2-3)
 *     vscan_merge                   cosine arg-max assignment + mean merge         (Eq. 4)
 *   Stage 2 (Sec. 4.2), at a middle LLM layer, per sequence:
 *     vscan_score (QK mode)         head mean of softmax(q_last . K) over a span   (Eq. 5)
 *     vscan_llm_prune               that score + top-k + compaction of hidden / K / V / position ids
 *
 * Conventions shared by every entry point
 *   - Returns a vscan_status.  Nothing throws, aborts or traps.  Arguments are validated on the
 *     host before any launch; on a validation error nothing is enqueued.
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, contiguous (row-major) in the
 *     layout stated, at least 16-byte aligned.  Inputs are only read.  Outputs must not overlap
 *     inputs.  NULL is allowed only where "optional" is written.
 *   - The library allocates no device memory and keeps no state between calls.  Scratch memory is
 *     a caller-provided `workspace` of at least vscan_*_workspace_bytes(desc) bytes, 256-byte
 *     aligned; its contents before the call are irrelevant and after the call unspecified.
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default stream) and
 *     is asynchronous with respect to the host; no call synchronises.
 *   - `dtype` is the element type of features, attention rows, q, K, V and hidden states
 *     (VSCAN_F32 or VSCAN_BF16).  Scores are always float32, indices int32.
 *   - Ties: wherever a top-k or an arg-max meets equal values the lowest index wins.  Survivor
 *     lists are in ascending original index.
 *   - Shapes are uniform over the batch of one call (mixed sizes: the *_ragged entry points).  Counts
 *     (k_global, k_per_window, k_keep) are explicit integers; percentages (R1, R2 of the paper) are
 *     resolved by the caller.
 */
#ifndef VSCAN_H_
#define VSCAN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define VSCAN_VERSION 100 /* major*10000 + minor*100 + patch */

typedef enum {
  VSCAN_OK = 0,
  VSCAN_ERR_INVALID_ARG = 1, /* null pointer, bad range, misalignment, overlap */
  VSCAN_ERR_UNSUPPORTED = 2, /* legal request this build cannot run (shape limit, dtype/path) */
  VSCAN_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
  VSCAN_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch error, no sm_100 device) */
  VSCAN_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out (reported by vscan_check) */
} vscan_status;

typedef enum { VSCAN_F32 = 0, VSCAN_BF16 = 1 } vscan_dtype;
typedef enum { VSCAN_SCORE_ROW = 0, VSCAN_SCORE_QK = 1, VSCAN_SCORE_RECEIVED = 2 } vscan_score_mode;
/* Eq. 5 takes the softmax over the visual keys only (SPAN_ONLY); Sec. 4.2's remark on recomputing
 * "vanilla attention" for the last token normalises over all keys (SPAN_FULL). */
typedef enum { VSCAN_SPAN_ONLY = 0, VSCAN_SPAN_FULL = 1 } vscan_softmax_span;
/* Which unit runs the similarity contraction of vscan_merge. */
typedef enum {
  VSCAN_MERGE_AUTO = 0,   /* bf16: TENSOR when the shape allows, else SIMT; f32: SIMT */
  VSCAN_MERGE_SIMT = 1,   /* fp32 FMA on CUDA cores (the only path for VSCAN_F32) */
  VSCAN_MERGE_TENSOR = 2, /* tcgen05 MMA, bf16 inputs, fp32 accumulation in tensor memory (kept sets above 128: the kept
                             rows are packed first and the MMAs run on CTA pairs); group sums in a second kernel, on
                             the tensor cores too (one-hot matrix products) where the shape allows */
  VSCAN_MERGE_CLUSTER = 3, /* assignment and group sums in ONE pass over the features: a cluster of dim / 256 CTAs per
                             instance, each owning 256 feature columns, exchanges partial dot products through
                             distributed shared memory (bf16, n_kept <= 64, dim 256 / 512 / 1024, no metric) */
  VSCAN_MERGE_INTERLEAVED = 4 /* the TENSOR path's two steps in one persistent launch, one CTA per SM: six warps
                             assign tile after tile (kept rows packed and their norms taken by a small
                             kernel first), eight more warps sum the groups of every instance whose tiles are
                             all done, reading its features from L2 (bf16, n_kept <= 256) */
} vscan_merge_path;

/* ---------------------------------------------------------------------------------------------
 * vscan_score
 *
 * ROW mode (Eq. 2): scores[b][j] = (1/heads) * sum_h attn[b][h][cls_offset + j], j in [0, n_tokens).
 *   attn      [instances][heads][row_len] of `dtype`: per-head attention probabilities of the [CLS]
 *             query (Eq. 1) or, for encoders without [CLS] (text after Eq. 2), the per-head attention
 *             each token receives, cls_offset = 0.  row_len >= cls_offset + n_tokens.
 *             The skipped entries are ignored; the row is not renormalised.
 *   scores    [instances][n_tokens] float32 (output).
 * QK mode (Eq. 5): for each query head h with KV head g = floor(h * kv_heads / q_heads),
 *   p_h = softmax_j(scale * q[b][h] . k[b][g][j]) taken over the span (SPAN_ONLY) or over all seq_len
 *   keys (SPAN_FULL); scores[b][j] = (1/q_heads) * sum_h p_h[span_begin + j], j in [0, span_len).
 *   q         [batch][q_heads][head_dim] of `dtype` (query of the last instruction token)
 *   k         [batch][kv_heads][seq_len][head_dim] of `dtype`
 *   scores    [batch][span_len] float32 (output).  head_dim must be a multiple of 8, at most 256;
 *             q_heads a multiple of kv_heads.
 * RECEIVED mode (Sec. 4.1, text after Eq. 2: encoders without [CLS] score a token by the average attention it
 *   receives from the other tokens): with P_h = softmax over keys of (scale * q[b][h] k[b][h]^T), row by row,
 *   r_h[j] = (1 / (seq_len - 1)) * sum_{i != j} P_h[i][j];  scores[b][j] = (1/q_heads) * sum_h r_h[j].
 *   The seq_len x seq_len matrix is never stored: two passes over 128 x 128 blocks on the tensor cores.
 *   q, k      [batch][q_heads][seq_len][head_dim] of `dtype` (kv_heads must equal q_heads)
 *   scores    [batch][seq_len] float32 (output)
 *   head_rows optional [batch][q_heads][seq_len] float32 output: the per-head r_h (what ROW mode takes as `attn`)
 *   This build: VSCAN_BF16 with head_dim 64 or 128, batch * q_heads <= 65535; else VSCAN_ERR_UNSUPPORTED.
 * Fields of the mode not in use are ignored.  Workspace: QK and RECEIVED modes.
 * Limits of this build (VSCAN_ERR_UNSUPPORTED, nothing enqueued): instances, batch <= 65535; QK mode:
 * (head_dim + keys under the softmax) * 4 bytes must fit 227 KB of shared memory (about 58 000 keys).
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  int32_t mode;  /* vscan_score_mode */
  int32_t dtype; /* vscan_dtype */
  /* ROW */
  const void* attn;
  int32_t instances, heads, row_len, cls_offset, n_tokens;
  /* QK */
  const void* q;
  const void* k;
  int32_t batch, q_heads, kv_heads, seq_len, head_dim, span_begin, span_len;
  int32_t softmax_span; /* vscan_softmax_span */
  float scale;
  /* output */
  float* scores;
  float* head_rows; /* RECEIVED mode, optional */
} vscan_score_desc;

size_t vscan_score_workspace_bytes(const vscan_score_desc* desc);
vscan_status vscan_score(const vscan_score_desc* desc, void* workspace, size_t workspace_bytes,
                         void* stream);

/* ---------------------------------------------------------------------------------------------
 * vscan_score_qk_static  (the paper has no counterpart: this is a packaging variant of the QK mode
 * above, same arithmetic, same result)
 *
 * For callers that cannot allocate device memory and therefore have no workspace to pass: code that
 * runs inside someone else's memory plan (an inference server whose pool is sized and frozen at
 * start-up, a plugin that is handed tensors but no allocator), or inside a region where
 * cudaMalloc is forbidden or would stall everything else on the GPU.  The call takes only the inputs
 * and the output; its scratch (the per-head probabilities, batch * q_heads * span_len floats) is a
 * fixed array built into the library, vscan_score_qk_static_capacity() floats long (1 Mi floats =
 * 4 MiB).  Every GPU on which the library is loaded carries those 4 MiB until the process exits.
 * The function calls no allocator of any kind.
 *   desc    a vscan_score_desc with mode = VSCAN_SCORE_QK; the fields mean what they mean above.
 *   Returns VSCAN_ERR_UNSUPPORTED when batch * q_heads * span_len exceeds the capacity (nothing is
 *   launched); the other statuses as for vscan_score.
 * The first call on a given device looks up the array's device address (one runtime query, cached per
 * device); make that first call outside any stream capture, with the target device current.
 * All calls on one GPU share the one array and it keeps whatever the last call left there.  A call
 * overwrites every entry it later reads, so stale contents are harmless and nothing needs clearing,
 * but two calls whose kernels overlap in time on the same GPU (different streams, or different host
 * threads) race on it and give wrong scores: keep calls on one stream, or order them yourself.
 * ------------------------------------------------------------------------------------------- */
size_t vscan_score_qk_static_capacity(void);
vscan_status vscan_score_qk_static(const vscan_score_desc* desc, void* stream);

/* ---------------------------------------------------------------------------------------------
 * vscan_select_global_local (Sec. 4.1, Eq. 2-3 and the footnote on duplicates)
 *
 * Tokens of an instance are numbered t = f*grid_h*grid_w + r*grid_w + c.  The grid is cut into
 * non-overlapping win_h x win_w windows (win_h | grid_h, win_w | grid_w).
 *   local scan : in every window the k_per_window tokens with the largest scores_local;
 *   global scan: the k_global largest scores_global among the tokens the local scan did not take;
 *   kept_idx   : the union, ascending, exactly K1 = windows*k_per_window + k_global per instance.
 *   scores_global, scores_local  [instances][N] float32, N = frames*grid_h*grid_w (may be the same
 *                                buffer)
 *   kept_idx   [instances][K1] int32 (output)
 *   kept_mask  [instances][N] uint8, 1 = kept (optional output)
 * Legal ranges: 0 <= k_per_window <= win_h*win_w, 0 <= k_global <= N - windows*k_per_window.
 * Limit of this build: N <= 16384.  No workspace needed (0 bytes).
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  const float* scores_global;
  const float* scores_local;
  int32_t instances, frames, grid_h, grid_w, win_h, win_w, k_per_window, k_global;
  int32_t* kept_idx;
  uint8_t* kept_mask;
} vscan_select_desc;

size_t vscan_select_workspace_bytes(const vscan_select_desc* desc);
vscan_status vscan_select_global_local(const vscan_select_desc* desc, void* workspace,
                                       size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * vscan_score_select (Eq. 2 and Eq. 3 in one launch)
 *
 * The same result as two ROW-mode vscan_score calls followed by vscan_select_global_local, without
 * the scores going through memory: the head means of attn_global / attn_local (layouts and meaning as
 * in vscan_score, ROW mode; the two may be the same buffer) are taken inside the selection kernel.
 *   select.scores_global / select.scores_local are here OPTIONAL OUTPUTS ([instances][N] float32)
 *   that receive the head means; every other field of `select` means what it means above.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  int32_t dtype; /* vscan_dtype of the attention rows */
  const void* attn_global;
  const void* attn_local;
  int32_t heads, row_len, cls_offset;
  vscan_select_desc select;
} vscan_score_select_desc;

vscan_status vscan_score_select(const vscan_score_select_desc* desc, void* stream);

/* ---------------------------------------------------------------------------------------------
 * vscan_merge (Sec. 4.1 "Token Merging", Eq. 4)
 *
 * For every token u not in kept_idx: a(u) = argmax_s cos(m_u, m_kept[s]) (lowest slot on ties; norms
 * clamped at 1e-12), where m is `metric` if given, else x.  Then
 *   merged[b][s] = (x_kept[s] + sum_{a(u)=s} x_u) / (1 + |{u : a(u)=s}|),
 * accumulated in float32 and rounded once to `dtype` (CUDA-core sums add in ascending token order; sums on
 * the tensor cores add tile by tile in the order of the hardware: the same result from run to run, not the
 * same last bit as the CUDA-core path).
 *   x         [instances][row_len][dim] of `dtype`; row cls_offset + t is token t; rows before
 *             cls_offset (the [CLS] feature) are never read.  row_len >= cls_offset + n_tokens.
 *   metric    optional [instances][row_len][metric_dim] of `dtype`
 *   kept_idx  [instances][n_kept] int32, strictly ascending, each in [0, n_tokens)  (not checked
 *             on the host; out-of-range entries are clamped on the device)
 *   merged    [instances][n_kept][dim] of `dtype` (output)
 *   assign    optional [instances][n_tokens] int32 output: slot of every token (a kept token maps
 *             to its own slot).  When NULL it lives in the workspace.
 *   counts    optional [instances][n_kept] int32 output: group size including the kept token.
 * dim and metric_dim must be multiples of 8; 1 <= n_kept <= n_tokens.
 * Limits of this build: n_tokens <= 29054 (one instance's member list is staged in shared memory),
 * instances <= 65535; beyond them VSCAN_ERR_UNSUPPORTED, nothing enqueued.
 * `path` picks the unit for the similarity contraction (vscan_merge_path).
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  int32_t dtype; /* vscan_dtype */
  int32_t path;  /* vscan_merge_path */
  const void* x;
  const void* metric;
  const int32_t* kept_idx;
  int32_t instances, row_len, cls_offset, n_tokens, dim, metric_dim, n_kept;
  void* merged;
  int32_t* assign;
  int32_t* counts;
} vscan_merge_desc;

size_t vscan_merge_workspace_bytes(const vscan_merge_desc* desc);
vscan_status vscan_merge(const vscan_merge_desc* desc, void* workspace, size_t workspace_bytes,
                         void* stream);

/* ---------------------------------------------------------------------------------------------
 * vscan_llm_prune (Sec. 4.2; KV-cache remark of the same section)
 *
 * The sequence is [n_sys system | n_vis visual | n_txt text] tokens, seq_len = n_sys+n_vis+n_txt.
 * Scores the visual span as vscan_score QK mode does (span_begin = n_sys, span_len = n_vis), keeps
 * the k_keep highest, and writes the shortened sequence of seq_out = seq_len - n_vis + k_keep rows:
 * system rows, surviving visual rows in ascending order, text rows.  Copies are bit-exact; position
 * ids keep their original values.
 *   q_last    [batch][q_heads][head_dim]           k, v   [batch][kv_heads][seq_len][head_dim]
 *   hidden    [batch][seq_len][hidden_dim]         pos_ids [pos_planes][batch][seq_len] int32
 *   kept_vis  [batch][k_keep] int32 output, indices relative to the visual span, ascending
 *   hidden_out [batch][seq_out][hidden_dim]        k_out, v_out [batch][kv_heads][seq_out][head_dim]
 *   pos_out   [pos_planes][batch][seq_out] int32
 *   scores    optional [batch][n_vis] float32 output
 * v/v_out, hidden/hidden_out and pos_ids/pos_out are optional as pairs (both NULL = skip).
 * hidden_dim*sizeof(dtype) and head_dim*sizeof(dtype) must be multiples of 16.  0 <= k_keep <= n_vis.
 * Limit of this build: n_vis <= 16384.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  int32_t dtype; /* vscan_dtype */
  const void* q_last;
  const void* k;
  const void* v;
  const void* hidden;
  const int32_t* pos_ids;
  int32_t batch, q_heads, kv_heads, head_dim, hidden_dim, pos_planes;
  int32_t n_sys, n_vis, n_txt, k_keep;
  int32_t softmax_span; /* vscan_softmax_span */
  float scale;
  int32_t* kept_vis;
  void* hidden_out;
  void* k_out;
  void* v_out;
  int32_t* pos_out;
  float* scores;
} vscan_prune_desc;

size_t vscan_llm_prune_workspace_bytes(const vscan_prune_desc* desc);
vscan_status vscan_llm_prune(const vscan_prune_desc* desc, void* workspace, size_t workspace_bytes,
                             void* stream);

/* ---------------------------------------------------------------------------------------------
 * Ragged batches (Sec. 5.1 "Models": encoders with dynamic resolution hand over between 4 and 16384 visual
 * tokens per image; Sec. 4.1 and 4.2 are per instance and per sequence, so units of different sizes are
 * independent problems).
 *
 * One call for instances (vscan_stage1_ragged: Eq. 2 + Eq. 3 selection, then the Eq. 4 merge) or sequences
 * (vscan_llm_prune_ragged: Sec. 4.2) whose sizes differ.  Every result is the one the uniform entry points give
 * for that unit alone.
 *   - The size, budget and offset arrays are HOST arrays with one entry per unit (the caller derives them from
 *     the image resolutions); they are read during the call and not kept.  Tensors are packed DEVICE buffers;
 *     unit i's block starts at the given ELEMENT offset of its buffer and has the uniform layout of that
 *     tensor for a batch of one.  Every block must start on a 16-byte boundary.
 *   - The library cuts the batch into runs of consecutive units with equal shape, equal budgets and regularly
 *     spaced blocks and enqueues the uniform kernels once per run on `stream`: a batch sorted by size costs
 *     one set of launches per distinct size, a batch of all-different sizes one set per unit.
 *   - Workspace: vscan_*_ragged_workspace_bytes(desc); vscan_check(workspace, stream) reports a bounded wait
 *     that ran out in any run.  Everything is validated before the first launch.
 * vscan_stage1_ragged
 *   attn_global, attn_local  per instance [heads][cls_offset + N_i] at attn_offset[i] (the two may be one buffer)
 *   x                        per instance [cls_offset + N_i][dim] at x_offset[i]
 *   kept_idx (out)           per instance [K1_i] at kept_offset[i], K1_i = windows_i * k_per_window[i] + k_global[i] >= 1
 *   merged (out)             per instance [K1_i][dim] at kept_offset[i] * dim
 *   N_i = frames[i] * grid_h[i] * grid_w[i] <= 16384; win_h | grid_h[i], win_w | grid_w[i]
 * vscan_llm_prune_ragged   (fields as in vscan_prune_desc, per sequence)
 *   q_last [batch][q_heads][head_dim] (uniform);  k, v per sequence [kv_heads][S_i][head_dim] at kv_offset[i];
 *   hidden [S_i][hidden_dim] at hidden_offset[i];  pos_ids [S_i] at pos_offset[i] (one plane);
 *   kept_vis (out) [k_keep[i]] at kept_offset[i];  k_out, v_out [kv_heads][S'_i][head_dim] at kv_out_offset[i];
 *   hidden_out [S'_i][hidden_dim] at hidden_out_offset[i];  pos_out [S'_i] at pos_out_offset[i];
 *   S_i = n_sys[i] + n_vis[i] + n_txt[i], S'_i = S_i - n_vis[i] + k_keep[i].  v / hidden / pos_ids optional as pairs.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
  int32_t dtype;      /* vscan_dtype */
  int32_t merge_path; /* vscan_merge_path */
  int32_t instances, heads, cls_offset, dim, win_h, win_w;
  const void* attn_global;
  const void* attn_local;
  const void* x;
  int32_t* kept_idx;
  void* merged;
  const int32_t* frames;       /* host arrays [instances] from here on */
  const int32_t* grid_h;
  const int32_t* grid_w;
  const int32_t* k_per_window;
  const int32_t* k_global;
  const int64_t* attn_offset;
  const int64_t* x_offset;
  const int64_t* kept_offset;
} vscan_stage1_ragged_desc;

size_t vscan_stage1_ragged_workspace_bytes(const vscan_stage1_ragged_desc* desc);
vscan_status vscan_stage1_ragged(const vscan_stage1_ragged_desc* desc, void* workspace, size_t workspace_bytes,
                                 void* stream);

typedef struct {
  int32_t dtype; /* vscan_dtype */
  int32_t batch, q_heads, kv_heads, head_dim, hidden_dim, pos_planes;
  int32_t softmax_span; /* vscan_softmax_span */
  float scale;
  const void* q_last;
  const void* k;
  const void* v;
  const void* hidden;
  const int32_t* pos_ids;
  int32_t* kept_vis;
  void* hidden_out;
  void* k_out;
  void* v_out;
  int32_t* pos_out;
  const int32_t* n_sys;        /* host arrays [batch] from here on */
  const int32_t* n_vis;
  const int32_t* n_txt;
  const int32_t* k_keep;
  const int64_t* kv_offset;
  const int64_t* kv_out_offset;
  const int64_t* hidden_offset;
  const int64_t* hidden_out_offset;
  const int64_t* pos_offset;
  const int64_t* pos_out_offset;
  const int64_t* kept_offset;
} vscan_prune_ragged_desc;

size_t vscan_llm_prune_ragged_workspace_bytes(const vscan_prune_ragged_desc* desc);
vscan_status vscan_llm_prune_ragged(const vscan_prune_ragged_desc* desc, void* workspace, size_t workspace_bytes,
                                    void* stream);

/* ---------------------------------------------------------------------------------------------
 * Housekeeping.
 * vscan_check: synchronises `stream` and reads the device status word at the start of a workspace
 * that the preceding call used; VSCAN_OK, VSCAN_ERR_TIMEOUT (a bounded wait expired) or
 * VSCAN_ERR_CUDA.  Only calls that take a non-empty workspace write that word.
 * vscan_last_cuda_error: cudaError_t value of the last failing runtime call on this thread (0 if none).
 * vscan_kernel_launches: number of kernels this library has launched in this process so far.
 * ------------------------------------------------------------------------------------------- */
int32_t vscan_version(void);
/* Per-kernel timing, a measurement aid with no counterpart in the paper.  Between
 * vscan_profile_begin(capacity) and vscan_profile_end every kernel the library launches is bracketed
 * by two CUDA events on its stream (up to `capacity` launches; later ones are not recorded).
 * vscan_profile_end waits for the recorded launches, writes for each, in launch order, a
 * NUL-terminated kernel name into names[i*32 .. i*32+31] and its duration in milliseconds into
 * millis[i] (both host arrays of `capacity` entries), releases the events and returns the count
 * (-1 if profiling was not on).  Do not use while a stream is being captured into a graph. */
vscan_status vscan_profile_begin(int32_t capacity);
int32_t vscan_profile_end(char* names, float* millis, int32_t capacity);
const char* vscan_status_string(vscan_status status);
vscan_status vscan_check(const void* workspace, void* stream);
int32_t vscan_last_cuda_error(void);
uint64_t vscan_kernel_launches(void);

/* ---------------------------------------------------------------------------------------------
 * vscan_selftest_bounded_wait: exercises the failure path of the device-side waits without touching any
 * data.  Visual rows of the Stage-2 compaction wait for their sequence's survivor list (Sec. 4.2, the
 * KV-cache remark: only survivors are moved) with a bound on the number of polls; when the bound runs out
 * the CTA records VSCAN_ERR_TIMEOUT in the status word and returns, and the context stays usable.  This call
 * launches one CTA that waits in the same way, `polls` polls of about 100 ns (1 .. 2^24), on a flag that
 * nothing sets; vscan_check(workspace, stream) must then return VSCAN_ERR_TIMEOUT.
 *   workspace  device memory, 256-byte aligned, at least 512 bytes; its first 512 bytes are overwritten.
 * ------------------------------------------------------------------------------------------- */
vscan_status vscan_selftest_bounded_wait(void* workspace, size_t workspace_bytes, uint32_t polls, void* stream);

/* ---------------------------------------------------------------------------------------------
 * vscan_selftest_fma_rate: a measurement aid with no counterpart in the paper.  Launches `blocks` CTAs of 256
 * threads that each run `iters` rounds of eight independent fp32 fused multiply-adds and stores `*flops`, the
 * floating-point operations of the launch (2 per FMA); the caller times the launch with events on `stream`.  The
 * rate is the ceiling that the CUDA-core similarity path of vscan_merge (VSCAN_MERGE_SIMT) is held against.
 *   scratch  device memory of at least blocks * 256 floats (overwritten)
 * ------------------------------------------------------------------------------------------- */
vscan_status vscan_selftest_fma_rate(float* scratch, size_t scratch_floats, int32_t blocks, int32_t iters, double* flops,
                                     void* stream);

#ifdef __cplusplus
}
#endif
#endif /* VSCAN_H_ */
