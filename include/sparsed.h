/*
 * sparsed.h - C ABI of the SparseD attention library for NVIDIA B200 (sm_100a).
 *
 * The library implements the attention hot path of SparseD (sparse attention for
 * diffusion language models): dense bidirectional attention for the early denoising
 * steps, a one-off per-head block-pattern selection at the switch step, and
 * block-sparse attention that reuses the pattern for all later steps (Algorithm 1).
 *
 * Conventions for every entry point
 *  - Pointers marked "device" are CUDA device pointers owned by the caller; the
 *    library never allocates or frees device memory and keeps no reference to caller
 *    buffers after a call returns. Pointers marked "host" are ordinary host pointers.
 *  - Tensors: Q and O are [batch, heads_q, seq_len, head_dim], K and V are
 *    [batch, heads_kv, seq_len, head_dim], bf16, head_dim contiguous. Strides for
 *    (batch, head, token) are given in elements; all-zero strides mean "contiguous".
 *    Base pointers must be 16-byte aligned and every stride a multiple of 8 elements.
 *    The fp32 side buffers (lse, tile_stats, scores, scores_out) and the workspace must be
 *    16-byte aligned too (the kernels read them with 16-byte loads), row_ptr and col_idx
 *    4-byte aligned; anything else is refused with SPARSED_ERR_ALIGNMENT before any launch.
 *    Output buffers (O, lse, tile_stats, scores_out, the pattern arrays) must not overlap any
 *    input of the same call: the kernels write them while other thread blocks still read.
 *  - Grouped-query attention: query head h reads key/value head h / (heads_q / heads_kv).
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *    stream) and return without synchronising. Argument problems are detected on the
 *    host before anything is launched and reported through the return code.
 *  - Every call takes a workspace `ws` (device) of at least
 *    sparsed_workspace_bytes(op, ...) bytes. Its first SPARSED_STATUS_BYTES bytes hold the
 *    device status word and must be zero before the first call (sparsed_workspace_init).
 *    Kernels never trap or spin forever: a wait that runs out records itself in the
 *    status word, which sparsed_last_device_status reads back.
 *  - Results are deterministic: the same inputs give bitwise the same outputs.
 */
#ifndef SPARSED_H_
#define SPARSED_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum sparsed_status {
  SPARSED_OK = 0,
  SPARSED_ERR_INVALID_ARG = 1,    /* null pointer, non-positive size, heads_q % heads_kv != 0, ... */
  SPARSED_ERR_UNSUPPORTED = 2,    /* head_dim != 128, block_size not in {32,64,128}, too many blocks */
  SPARSED_ERR_ALIGNMENT = 3,      /* seq_len or prefill_len not a multiple of block_size; pointer/stride alignment */
  SPARSED_ERR_WORKSPACE = 4,      /* workspace missing or too small */
  SPARSED_ERR_PATTERN = 5,        /* pattern arrays missing, too small, or inconsistent with the shape */
  SPARSED_ERR_ARCH = 6,           /* current device is not compute capability 10.x */
  SPARSED_ERR_CUDA = 7,           /* a CUDA call failed; see sparsed_last_cuda_error() */
  SPARSED_ERR_DEVICE_TIMEOUT = 8  /* a bounded device-side wait ran out (from the status word) */
} sparsed_status;

#define SPARSED_STATUS_BYTES 256

/* Operation ids for sparsed_workspace_bytes. */
#define SPARSED_OP_ATTN_FULL 0
#define SPARSED_OP_SELECT_PATTERN 1
#define SPARSED_OP_SELECT_FROM_SCORES 2
#define SPARSED_OP_ATTN_SPARSE 3
#define SPARSED_OP_PATTERN_VALIDATE 4
#define SPARSED_OP_SELECT_POOLED_QK 5
#define SPARSED_OP_ATTENTION_STEP 6

/* Schedule modes returned by sparsed_schedule_mode. */
#define SPARSED_MODE_FULL 0
#define SPARSED_MODE_FULL_AND_SELECT 1
#define SPARSED_MODE_SPARSE 2

typedef struct sparsed_shape {
  int32_t batch, heads_q, heads_kv, seq_len, head_dim;
  int64_t q_strides[3], k_strides[3], v_strides[3], o_strides[3]; /* elements: batch, head, token */
  float softmax_scale;                                            /* 0 => 1/sqrt(head_dim) */
} sparsed_shape;

typedef struct sparsed_select_params {
  int32_t block_size;  /* 32, 64 or 128 (the paper uses 32 for short and 128 for long contexts) */
  int32_t prefill_len; /* p of Eq. 6: keys [0,p) are prefill, [p,seq_len) generation; multiple of block_size */
  double keep_ratio;   /* rho in (0,1] */
  int32_t rounding;    /* 0: kept = ceil(rho * blocks in region) (default), 1: floor; at least 1 */
} sparsed_select_params;

/* Block pattern of Eq. 4 as CSR lists: row r = (b*heads_q + h)*num_blocks + query_block;
 * col_idx[row_ptr[r] .. row_ptr[r+1]) are the kept key blocks, strictly ascending. */
typedef struct sparsed_pattern {
  int32_t *row_ptr;     /* device, batch*heads_q*num_blocks + 1 entries */
  int32_t *col_idx;     /* device, col_capacity entries */
  int64_t col_capacity; /* entries available in col_idx */
  int64_t nnz;          /* set by the selection calls: entries used */
  int32_t block_size, num_blocks, batch, heads_q; /* set by the selection calls */
} sparsed_pattern;

/*
 * Dense bidirectional attention, O = softmax(Q K^T / sqrt(d)) V with no mask (Eq. 1 and
 * the "A(Q,K) V" of Section 3.1; the full-attention branch of Algorithm 1).
 * q,k,v,o: device bf16. lse_or_null: device fp32 [batch, heads_q, seq_len] receiving the
 * natural-log sum of exponentials of each query row's scaled logits, or NULL.
 * Any seq_len >= 1 is accepted. Errors: INVALID_ARG, UNSUPPORTED (head_dim != 128),
 * ALIGNMENT, WORKSPACE, ARCH, CUDA.
 */
sparsed_status sparsed_attn_full(const sparsed_shape *shape, const void *q, const void *k, const void *v,
                                 void *o, float *lse_or_null, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Pattern selection at the switch step ("Isolated Selection", Eq. 5 and Eq. 6, the inner
 * loop of Algorithm 1): A' = avgpool(softmax(Q K^T / sqrt(d)), block_size) is computed one
 * query block at a time without materialising the l x l matrix; for each head and query
 * block the top-rho% key blocks are chosen separately among prefill and generation blocks,
 * ranked by A' (fp32), ties to the lower block index, and written as ascending CSR lists.
 * lse_or_null: the LSE written by sparsed_attn_full for the same Q,K (saves a pass), or NULL.
 * scores_out_or_null: device fp32 [batch, heads_q, nb, nb] receiving A', or NULL (then the
 * workspace holds it). `out`: host struct; its row_ptr/col_idx/col_capacity are inputs, the
 * other fields are filled in. Requires seq_len % block_size == 0 and
 * prefill_len % block_size == 0. Errors: as above plus PATTERN (capacity too small).
 */
sparsed_status sparsed_select_pattern(const sparsed_shape *shape, const sparsed_select_params *params,
                                      const void *q, const void *k, const float *lse_or_null,
                                      sparsed_pattern *out, float *scores_out_or_null, void *ws,
                                      size_t ws_bytes, void *cuda_stream);

/*
 * The ranking half of the selection alone (Eq. 5 / Eq. 6 applied to a given A'):
 * scores: device fp32 [batch, heads_q, num_blocks, num_blocks]. NaN scores rank lowest.
 */
sparsed_status sparsed_select_from_scores(const sparsed_select_params *params, const float *scores,
                                          int32_t batch, int32_t heads_q, int32_t num_blocks,
                                          sparsed_pattern *out, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The switch step without a second Q K^T pass. Algorithm 1 runs full attention at the switch
 * step and then computes A' = avgpool(A) from the same Q and K; A' can be formed from row
 * statistics of that very full-attention pass:
 *   sparsed_attn_full_stats   = sparsed_attn_full that also records, for every query row and
 *                               every key block of `block_size` keys (32, 64 or 128: the block size
 *                               the pattern will be selected with), log2 of the block's share of the
 *                               row's softmax denominator (tile_stats, device fp32,
 *                               sparsed_tile_stats_bytes() bytes, layout
 *                               [batch*heads_q][ceil(seq_len/128)][seq_len/block_size][128]:
 *                               128-row query tile, key block, row in the query tile);
 *                               lse is required here; seq_len must be a multiple of block_size.
 *   sparsed_select_from_stats = pools those statistics into A' (2^(stat - LSE) is the
 *                               probability mass a row puts on a key block), ranks it as
 *                               sparsed_select_pattern does (Eq. 5 / Eq. 6) and writes the CSR
 *                               pattern; scores_out_or_null optionally receives A'.
 *                               params->block_size must be the block size the statistics were
 *                               recorded with.
 * Same rules and errors as sparsed_attn_full / sparsed_select_pattern; the selection needs
 * seq_len / block_size <= 2048 (UNSUPPORTED beyond). Both buffers are caller-owned device memory.
 * sparsed_attn_full_stats runs on a kernel whose MMAs span pairs of CTAs (launched as clusters of two);
 * sparsed_attn_full runs on it from 16384 tokens on and on a single-CTA kernel below that. The environment
 * variable SPARSED_DENSE_KERNEL=pair|single, read at the first call, sends sparsed_attn_full to one of
 * them at every length, for measurements.
 */
sparsed_status sparsed_tile_stats_bytes(const sparsed_shape *shape, int32_t block_size,
                                        size_t *out_bytes); /* host only */
sparsed_status sparsed_attn_full_stats(const sparsed_shape *shape, int32_t block_size, const void *q,
                                       const void *k, const void *v, void *o, float *lse, float *tile_stats,
                                       void *ws, size_t ws_bytes, void *cuda_stream);
sparsed_status sparsed_select_from_stats(const sparsed_shape *shape, const sparsed_select_params *params,
                                         const float *lse, const float *tile_stats, sparsed_pattern *out,
                                         float *scores_out_or_null, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Block-mean ESTIMATE of A' and the selection from it. NOT the paper's scorer: the paper pools the
 * exact post-softmax probabilities; this is the cheaper kind of estimate (pool first, then score)
 * that the introduction sets the method against, offered so that its recall of the exact pattern
 * and its cost can be measured on the same inputs through the same selection (Eq. 5 / Eq. 6):
 *   mean_q[i], mean_k[j] = means of the rows of query block i / key block j (fp32),
 *   est[i][j] = softmax_j(softmax_scale * mean_q[i] . mean_k[j]) / block_size
 * (rows sum to 1 / block_size like A'; equal to A' when every block is constant).
 * q, k: device bf16, layouts and strides as for sparsed_attn_full (v/o strides ignored).
 * out: caller-owned CSR buffers as for sparsed_select_pattern; scores_out_or_null optionally
 * receives est (device fp32 [batch, heads_q, num_blocks, num_blocks]).
 * Workspace: sparsed_workspace_bytes(SPARSED_OP_SELECT_POOLED_QK, shape, params) bytes (status
 * block + the block means). block_size 32, 64 or 128; seq_len / block_size <= 1024
 * (UNSUPPORTED beyond). Asynchronous on the stream; deterministic.
 */
sparsed_status sparsed_select_pattern_pooled_qk(const sparsed_shape *shape, const sparsed_select_params *params,
                                                const void *q, const void *k, sparsed_pattern *out,
                                                float *scores_out_or_null, void *ws, size_t ws_bytes,
                                                void *cuda_stream);

/*
 * Block-sparse attention, O = softmax((Q K^T + M_S) / sqrt(d)) V with M_S the 0 / -inf block
 * mask given by `pattern` (Eq. 3 and Eq. 4; the "Sparse Reusing" branch of Algorithm 1).
 * Accepts any CSR whose rows are ascending and in range (not only selected ones); a query
 * block with an empty list gets zeros. Requires seq_len == pattern->num_blocks *
 * pattern->block_size; with 64- or 32-key blocks at most 2048 blocks per row (UNSUPPORTED
 * beyond). Errors: as above plus PATTERN.
 */
sparsed_status sparsed_attn_sparse(const sparsed_shape *shape, const sparsed_pattern *pattern, const void *q,
                                   const void *k, const void *v, void *o, void *ws, size_t ws_bytes,
                                   void *cuda_stream);

/*
 * Step schedule ("Skipping Sparse", the outer branch of Algorithm 1). Steps are 1-based.
 * The switch step is s = clamp(floor(total_steps * skip), 1, total_steps); steps before s
 * are FULL, step s is FULL_AND_SELECT (full attention, then select), later steps SPARSE.
 * Host only. sparsed_schedule_mode returns a SPARSED_MODE_* value or -1 on bad arguments;
 * sparsed_switch_step returns s or -1.
 */
int32_t sparsed_schedule_mode(int32_t step_1based, int32_t total_steps, double skip);
int32_t sparsed_switch_step(int32_t total_steps, double skip);

/*
 * Algorithm 1 for one attention call of denoising step `step_1based` (1-based) of `total_steps`:
 *   steps before the switch step  : full attention (Eq. 1)                  -> *mode = SPARSED_MODE_FULL
 *   the switch step               : full attention, then the pattern is selected from that very pass
 *                                   (A' = avgpool(A), Eq. 5 / Eq. 6) and written to `pattern`
 *                                                                            -> SPARSED_MODE_FULL_AND_SELECT
 *   later steps                   : block-sparse attention (Eq. 3 / Eq. 4) with `pattern` as the
 *                                   switch step left it ("Sparse Reusing")   -> SPARSED_MODE_SPARSE
 * The same calls as sparsed_attn_full / sparsed_attn_full_stats + sparsed_select_from_stats /
 * sparsed_attn_sparse, chosen by sparsed_schedule_mode; where the statistics path does not apply
 * (more than 2048 key blocks per row) the switch step selects with sparsed_select_pattern instead.
 * q, k, v, o: device bf16 as for sparsed_attn_full. pattern: caller-owned CSR buffers sized as for
 * sparsed_select_pattern, written at the switch step and only read afterwards; the caller keeps it
 * (one per layer) across steps. ws: device workspace, zeroed status block first; the switch step
 * needs sparsed_workspace_bytes(SPARSED_OP_ATTENTION_STEP, shape, params) bytes (row statistics of
 * the full pass: about 4 * seq_len * seq_len / block_size bytes per head), every other step only
 * SPARSED_STATUS_BYTES. mode_out_or_null (host) receives the mode that ran. Errors as for the calls
 * it makes; INVALID_ARG for a step outside 1..total_steps or skip outside [0, 1]. Asynchronous.
 */
sparsed_status sparsed_attention_step(const sparsed_shape *shape, const sparsed_select_params *params,
                                      int32_t step_1based, int32_t total_steps, double skip, const void *q,
                                      const void *k, const void *v, void *o, sparsed_pattern *pattern, void *ws,
                                      size_t ws_bytes, void *cuda_stream, int32_t *mode_out_or_null);

/*
 * sparsed_attention_step with one of the method's components switched off: the rows of the paper's
 * component ablation (Table 2) as modes of the same call, for timing and for comparison.
 *   SPARSED_VARIANT_NO_REUSE     "- Sparse Reusing": every sparse step first selects its own pattern from
 *                                that step's Q and K (sparsed_select_pattern with no LSE: a row-statistics
 *                                pass, pooled scoring, ranking) and then attends on it; `pattern` is
 *                                overwritten at every sparse step. Such steps need
 *                                sparsed_workspace_bytes(SPARSED_OP_SELECT_PATTERN, ...) bytes of workspace.
 *   SPARSED_VARIANT_NO_ISOLATION "- Isolated Selection": prefill_len is ignored, one top-rho% over all key
 *                                blocks (Eq. 5 without the split of Eq. 6).
 * ("- Skipping Sparse" is skip = 0: the first step is the switch step.) Flags may be combined; 0 is
 * sparsed_attention_step itself. Everything else as for sparsed_attention_step; INVALID_ARG for
 * unknown flag bits.
 */
#define SPARSED_VARIANT_NO_REUSE 1
#define SPARSED_VARIANT_NO_ISOLATION 2
sparsed_status sparsed_attention_step_variant(const sparsed_shape *shape, const sparsed_select_params *params,
                                              int32_t variant, int32_t step_1based, int32_t total_steps,
                                              double skip, const void *q, const void *k, const void *v, void *o,
                                              sparsed_pattern *pattern, void *ws, size_t ws_bytes,
                                              void *cuda_stream, int32_t *mode_out_or_null);

/*
 * Number of key blocks kept per query block in the prefill and generation regions
 * (Eq. 6's "top-rho%" counted in blocks). Host only; k_pre / k_gen are host pointers.
 */
sparsed_status sparsed_kept_per_row(const sparsed_select_params *params, int32_t seq_len, int32_t *k_pre,
                                    int32_t *k_gen);

/* Workspace size in bytes for one SPARSED_OP_*; `shape`/`params` may be NULL where unused. Host only. */
sparsed_status sparsed_workspace_bytes(int32_t op, const sparsed_shape *shape,
                                       const sparsed_select_params *params, size_t *out_bytes);

/* Zeroes the status block of a workspace (asynchronous memset on the stream). */
sparsed_status sparsed_workspace_init(void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Fixed comparison patterns in the same CSR form (the sliding-window and sink-plus-window
 * baselines of the paper's "Experimental Setting", expressed in blocks): query block i keeps the
 * key blocks [0, sink_blocks) and those with |j - i| <= (window_blocks - 1) / 2 (a symmetric
 * window, since the attention is bidirectional). Lists are ascending; rows near the edges are
 * shorter. `out`: row_ptr/col_idx/col_capacity are inputs (capacity is checked against the exact
 * count, returned in nnz). Device arrays are written asynchronously on the stream.
 */
sparsed_status sparsed_build_window_pattern(int32_t batch, int32_t heads_q, int32_t num_blocks, int32_t block_size,
                                            int32_t sink_blocks, int32_t window_blocks, sparsed_pattern *out,
                                            void *cuda_stream);

/*
 * Checks a pattern on the device: row_ptr monotone and within capacity, every list strictly
 * ascending and within [0, num_blocks), no empty row. Synchronises the stream. Returns
 * SPARSED_OK or SPARSED_ERR_PATTERN. (No paper counterpart: a guard for user-built masks.)
 */
sparsed_status sparsed_pattern_validate(const sparsed_pattern *pattern, void *ws, size_t ws_bytes,
                                        void *cuda_stream);

/* Reads the device status word (synchronises the stream). code 0 = fine, 1 = a bounded wait ran out
 * (`where` identifies the wait), 2 = a kernel found its shared memory misaligned, 3 = sparsed_attn_sparse
 * met a row_ptr entry that points outside col_idx (that query block's rows were written as zeros),
 * 4 = the two CTAs of a pair in sparsed_attn_full_stats got different tensor-memory bases (the pair did no
 * work). Returns SPARSED_ERR_DEVICE_TIMEOUT if code != 0. */
sparsed_status sparsed_last_device_status(void *ws, void *cuda_stream, int32_t *code, int32_t *where);

/*
 * sparsed_select_pattern for callers that cannot give it a workspace because they cannot
 * allocate device memory at this point: for example a serving process whose own pool took
 * all of the GPU's memory at start-up (a later cudaMalloc would fail), or a request path
 * on which allocation is banned because cudaMalloc and cudaFree stall the whole device.
 * (The paper has no counterpart; this is a deployment convenience.)
 *
 * Same inputs, outputs, rules and errors as sparsed_select_pattern with scores_out = NULL,
 * but the scratch (status block, pooled scores, and the LSE rows if lse_or_null is NULL)
 * is a fixed array of SPARSED_STATIC_SCRATCH_BYTES inside the library's device image, which
 * every GPU that loads the library holds until the process exits. The call allocates and
 * frees nothing, on the device or through any library.
 *  - Limit: sparsed_workspace_bytes(SPARSED_OP_SELECT_PATTERN, ...) minus the LSE part when
 *    an LSE is passed must not exceed SPARSED_STATIC_SCRATCH_BYTES, else the call returns
 *    SPARSED_ERR_WORKSPACE and launches nothing (use sparsed_select_pattern instead).
 *  - The first call on each device looks up the array's device address (with that device
 *    current); make that first call before any stream capture begins.
 *  - All calls on a device share the one array: calls that can overlap on the GPU (different
 *    streams, different threads) race on it. Serialise them. The array keeps the previous
 *    call's contents; the call itself re-zeroes the part that has to start at zero.
 *  - Device-side wait timeouts of this variant are recorded in the internal array, which
 *    sparsed_last_device_status cannot read; check the pattern with sparsed_pattern_validate
 *    if in doubt.
 */
#define SPARSED_STATIC_SCRATCH_BYTES (8u << 20)
sparsed_status sparsed_select_pattern_static(const sparsed_shape *shape, const sparsed_select_params *params,
                                             const void *q, const void *k, const float *lse_or_null,
                                             sparsed_pattern *out, void *cuda_stream);

/*
 * Self-test of the failure path (no paper counterpart): launches one warp that waits, with a short
 * poll limit, on a barrier nothing completes. The wait gives up, the kernel returns normally, and
 * the status word of `ws` then reads code 1, where 99 (sparsed_last_device_status returns
 * SPARSED_ERR_DEVICE_TIMEOUT). Clear it with sparsed_workspace_init; the context stays usable.
 */
sparsed_status sparsed_selftest_wait_timeout(void *ws, size_t ws_bytes, void *cuda_stream);

const char *sparsed_status_string(sparsed_status status);
int32_t sparsed_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SPARSED_H_ */
