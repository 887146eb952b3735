/*
 * liblsa — C ABI of the LongCat-Sparse-Attention indexer + sparse-attention forward
 * for NVIDIA B200 (sm_100a).
 *
 * The path (one cross-layer group of R attention layers that share one index set):
 *
 *   a0  lsa_block_means   sub-block mean keys                       Sec. 3.3, stage 1 (first paragraph)
 *   a1  coarse page score I_page[t,p]                               Eq. 9
 *   a2  top-M pages                                                 Eq. 10
 *   a3  fine token score  I[t,s] on the recalled pages              Eq. 11 (= Eq. 1)
 *   a4  top-K_sparse outside sink and window                        Eq. 12 with Eq. 6-7
 *   a5  lsa_convert       index set -> contiguous pieces / physical cache rows   Sec. 3.1 (streaming-aware layout)
 *   a6  lsa_sparse_attn   attention over sink U window U sparse     Eq. 3, Sec. 4.1.1
 *   a7  lsa_layer_group   a0..a5 once, a6 for each of the R layers  Sec. 3.2
 *
 * Conventions
 *   - Positions are 0-indexed.  Query t sees keys s <= t.  S = k_sink, W = k_swa, Ksp = k_sparse.
 *     Candidate range of query t: C(t) = [S, t-W] (empty when t-W < S).  sink = [0, min(S,t+1)),
 *     window = [max(S, t-W+1), t].
 *   - Every pointer is a DEVICE pointer owned by the caller unless its comment says "host".
 *     The library allocates no device memory: scratch lives in the workspace given to
 *     lsa_create (size it with lsa_workspace_bytes).
 *   - Every call enqueues work on the context's stream and returns without waiting.
 *   - Return value: LSA_OK or a negative lsa_error.  Nothing throws, aborts or traps.
 *     A device-side status word (0 = fine) records kernel-detected problems (bounded wait
 *     expired); read it with lsa_status.
 *   - bf16 tensors are passed as void*; rows are contiguous unless a leading dimension is given.
 *     All base pointers must be 16-byte aligned and every row stride a multiple of 16 bytes.
 *   - Top-K order is total: larger score first, on equal scores the smaller position first;
 *     +0 and -0 are equal.  Inputs must be finite.  Selected positions are reported ascending.
 *
 * Supported shapes (anything else returns LSA_ERR_SHAPE):
 *   indexer  (H_I, d_I) in {(8,64), (64,128)};  page P in {64,128,256}, sub_block B with P/B in
 *            {8,16,32};  k_sparse <= 4096, multiple of 4;  recall budget keep_pages*P <= 4096, or, for the
 *            (64,128) indexer on contiguous caches, any multiple of 128 up to 262144 (the candidates' scores
 *            then pass through the workspace: 4 bytes per candidate and query of a pass, see q_chunk)
 *   attention (H, d_qk, d_v) in {(16,128,128), (64,576,512)}
 *   paged mode needs kv_page == page.
 */
#ifndef LSA_H_
#define LSA_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LSA_API __attribute__((visibility("default")))
#else
#define LSA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LSA_OK = 0,
  LSA_ERR_ARG = -1,        /* null pointer, negative size, inconsistent arguments */
  LSA_ERR_SHAPE = -2,      /* dimension or alignment the kernels do not support */
  LSA_ERR_WORKSPACE = -3,  /* workspace missing or smaller than lsa_workspace_bytes says */
  LSA_ERR_CUDA = -4,       /* a CUDA runtime call failed (see lsa_last_cuda_error) */
  LSA_ERR_TIMEOUT = -5,    /* a bounded device-side wait expired (reported through lsa_status) */
  LSA_ERR_CAPACITY = -6,   /* the call needs more scratch than a fixed-capacity entry point owns */
  LSA_ERR_INDEX = -7       /* checking build only (library compiled with -DLSA_CHECK, `python -m
                              paper_2608_01662_b200.build --check`): an attention kernel met a cache row number
                              outside [0, n_key) in a caller-given sparse list or row list; the row was skipped (it
                              contributes nothing) and the code is reported through lsa_status.  The normal build
                              trusts these lists, as it trusts its pointers */
} lsa_error;

enum { LSA_KEY_BF16 = 0, LSA_KEY_E4M3 = 1 };

typedef struct lsa_ctx lsa_ctx;

/* Plain data; set struct_size = sizeof(lsa_params). */
typedef struct {
  uint32_t struct_size;
  int32_t n_heads_idx;  /* H_I  (Eq. 1) */
  int32_t d_idx;        /* d_I */
  int32_t key_dtype;    /* LSA_KEY_BF16, or LSA_KEY_E4M3 = OCP e4m3 codes + one fp32 scale per token */
  int32_t page;         /* P   (Sec. 3.3) */
  int32_t sub_block;    /* B,  divides P */
  int32_t keep_pages;   /* M */
  int32_t k_sparse;     /* Ksp (Eq. 6) */
  int32_t k_sink;       /* S */
  int32_t k_swa;        /* W */
  int32_t n_heads;      /* H  attention heads; all share one K/V row per token (absorbed MQA, Sec. 2.2) */
  int32_t d_qk;
  int32_t d_v;
  float sm_scale;       /* logits = sm_scale * q.k */
  int32_t n_layers;     /* R, size of the cross-layer group (Sec. 3.2) */
  int32_t q_chunk;      /* queries scored per pass of the indexer in lsa_layer_group; 0 = all at once */
  int32_t hi_enable;    /* 1: two-stage selection (Eq. 9-12); 0: every eligible page is kept (Eq. 7) */
  int32_t paged;        /* 0: caches are [n_key, d] arrays and queries are consecutive positions (prefill)
                           1: caches are pools [n_phys_pages*kv_page, d] read through page_table and there is
                              one query per sequence at position ctx_len[b]-1 (decode) */
  int32_t kv_page;      /* tokens per physical cache page (paged mode) */
  int32_t pooling;      /* coarse-stage pooling of a sub-block: LSA_POOL_MEAN (Eq. 9, the paper's choice) or
                           LSA_POOL_MINMAX (Eq. 13, the variant of its pooling ablation; contiguous caches only) */
} lsa_params;

enum { LSA_POOL_MEAN = 0, LSA_POOL_MINMAX = 1 };

/* ---- context ------------------------------------------------------------------------------ */

/* Create a context bound to `device` and to `cuda_stream` (a cudaStream_t; NULL = legacy default).
 * `workspace` is caller-owned device memory of `workspace_bytes` bytes, 256-byte aligned, that must
 * outlive the context; calls on one context must not overlap on the GPU.  Host allocations only. */
LSA_API int lsa_create(lsa_ctx** ctx, int device, void* cuda_stream, void* workspace, size_t workspace_bytes);
LSA_API int lsa_destroy(lsa_ctx* ctx);

/* Scratch needed by any call with these parameters for n_query queries (prefill: the largest number
 * passed to one call; with q_chunk > 0 lsa_layer_group needs only q_chunk of them), caches of at most
 * n_key_max tokens per sequence and `batch` sequences (paged mode).  Writes *bytes (host). */
LSA_API int lsa_workspace_bytes(const lsa_params* p, int64_t n_query, int64_t n_key_max, int batch, size_t* bytes);

/* Waits for the stream, then writes the device status word (host int; 0 = fine, LSA_ERR_TIMEOUT...)
 * and clears it. */
LSA_API int lsa_status(lsa_ctx* ctx, int* device_status);

/* Failure-detection self-test.  Launches one small block whose threads wait, as every tcgen05 kernel of the library
 * waits, on a shared-memory barrier - but one that nobody ever arrives on.  Thread 0 gives up after `budget_cycles`
 * SM clock cycles (at most 2^31, about a second) and records LSA_ERR_TIMEOUT in the context's status word; the other
 * threads see the word and stop; the kernel ends normally.  Afterwards lsa_status reports LSA_ERR_TIMEOUT (and
 * clears it) and the context serves further calls as before.  Nothing faults, traps or hangs.
 * (The paper has no counterpart: this exercises the library's own handling of a wait that runs out.) */
LSA_API int lsa_selftest_wait(lsa_ctx* ctx, int64_t budget_cycles);
LSA_API const char* lsa_strerror(int err);
/* Text of the last CUDA error seen by this context (host string owned by the library). */
LSA_API const char* lsa_last_cuda_error(lsa_ctx* ctx);
/* Number of kernels this context has launched since creation (host counter). */
LSA_API int64_t lsa_launch_count(lsa_ctx* ctx);

/* Launch-shape knobs; results never depend on them.
 *   LSA_TUNE_COARSE_GROUPS  4-query groups held per thread block of the coarse-score kernel (1 or 2; default 2)
 *   LSA_TUNE_ATTN_TC        1 (default): MLA-shape attention on tcgen05.mma; 0: the mma.sync kernel
 *   LSA_TUNE_ATTN_SPLIT     row splits per sequence in paged attention: 0 (default) = chosen by the wave cost model,
 *                           1..16 = fixed (the tcgen05 kernel merges its splits inside a thread-block cluster and
 *                           accepts 1, 2, 4 or 8; other values make lsa_sparse_attn return LSA_ERR_ARG there)
 *   LSA_TUNE_ATTN_PV_WAIT   prefill on the tcgen05 attention kernel.  0 (default): the Q K^T of a tile follows the P V that
 *                           frees its accumulator in the issuing thread's program order; 1: it waits for that P V's
 *                           completion barrier (slower, same bits).  Paged calls always wait.
 *   LSA_TUNE_ATTN_GATHER    tcgen05 attention kernel, scattered cache rows.  0 (default): coalesced 16-byte cp.async
 *                           copies; 1: TMA gather, four rows per cp.async.bulk.tensor tile::gather4 instruction (needs a
 *                           16-byte aligned cache whose row pitch is a multiple of 16 bytes, else the other path is
 *                           taken).  Same bits; the TMA path measured 1.3 x slower (512 bytes per instruction).
 *   LSA_TUNE_FINE_PAGED_TC  hierarchical indexer on paged caches, fine stage (64-head indexer, 64-token pages; other
 *                           shapes always take form 2).  0 (default): one kernel, a thread-block cluster per sequence:
 *                           page top-M, token scores of the kept pages on tcgen05, top-K and cache rows; 1: the same
 *                           steps as three kernels (page lists, the scoring kernel the flat paged indexer uses,
 *                           top-K); 2: page top-M and token scores in one mma.sync kernel, several blocks per
 *                           sequence, then a top-K kernel.  Same selection.  cfg4: 33 / 72 / 58 us per decode step. */
enum { LSA_TUNE_COARSE_GROUPS = 0, LSA_TUNE_ATTN_TC, LSA_TUNE_ATTN_SPLIT, LSA_TUNE_ATTN_PV_WAIT, LSA_TUNE_ATTN_GATHER,
       LSA_TUNE_FINE_PAGED_TC, LSA_TUNE_COUNT };
LSA_API int lsa_tune(lsa_ctx* ctx, int knob, int value);

/* Per-kernel timing.  While enabled, every kernel-launching call records a CUDA event pair on the
 * context's stream around the launches of each kernel class (at most 4096 pairs between reads; later
 * launches go unrecorded).  lsa_profile_read waits for the stream and writes, per class, the summed
 * device time in ms and the number of recorded launches (host arrays of LSA_K_COUNT entries), then
 * starts over.  The first enable creates the events (host resources only). */
/* lsa_append is timed as LSA_K_MEANS */
enum { LSA_K_MEANS = 0, LSA_K_COARSE, LSA_K_FINE_SELECT, LSA_K_SELECT, LSA_K_CONVERT, LSA_K_ATTN, LSA_K_MERGE, LSA_K_COUNT };   /* lsa_merge is timed as LSA_K_MERGE */
LSA_API int lsa_profile_enable(lsa_ctx* ctx, int on);
LSA_API int lsa_profile_read(lsa_ctx* ctx, double* total_ms, int64_t* launches);

/* ---- a0: mean-key cache (Sec. 3.3) ---------------------------------------------------------- */

/* kmean[n, :] = mean over the tokens present in sub-block n of the (dequantised) indexer keys, fp32
 * accumulation, stored bf16 (round to nearest even).
 *   k_idx    bf16 [n_key, d_I]  or  uint8 e4m3 codes [n_key, d_I] with k_scale fp32 [n_key]
 *   kmean    bf16 [ceil(n_key/B), d_I]
 * Paged mode: k_idx / k_scale are pools indexed by physical row and kmean is the twin pool
 * [n_phys_pages*kv_page/B, d_I]: sub-block j of physical page g is row g*(kv_page/B)+j.  The means of
 * sequence b's first ctx_len[b] tokens are written (a trailing partial sub-block averages the tokens
 * present); n_key is ignored; page_table int32 [batch, page_table_stride].
 * Prefill: page_table = ctx_len = NULL, batch = 1.
 * With pooling = LSA_POOL_MINMAX (Sec. 5, "Pooling method") the cache holds the per-dimension extrema instead:
 *   kmean    bf16 [ceil(n_key/B), 2*d_I]: row n = [max over the sub-block's tokens | min over them], each value
 *            the dequantised key value rounded to bf16; paged mode returns LSA_ERR_SHAPE. */
LSA_API int lsa_block_means(lsa_ctx* ctx, const lsa_params* p, const void* k_idx, const float* k_scale,
                    int64_t n_key, const int32_t* page_table, int64_t page_table_stride,
                    const int32_t* ctx_len, int batch, void* kmean);

/* Cache maintenance of one decode step (paged mode only; Sec. 3.3 keeps the mean keys with the cache, Sec. 4.1
 * lists their upkeep among the costs of decoding): for every sequence b the new token's indexer key is stored at
 * position ctx_len[b] and the mean of the sub-block holding that position is recomputed over the tokens now present
 * (the same arithmetic as lsa_block_means, so an appended cache equals a rebuilt one bit for bit).
 *   k_new    bf16 [batch, d_I]: the new indexer keys.  For e4m3 caches each is quantised here: scale = amax / 448
 *            (1 for a zero row), code = round-to-nearest-even of k / scale in fp32, saturating.
 *   k_idx / k_scale / kmean   the pools of lsa_block_means, written in place
 *   ctx_len  int32 [batch]: lengths BEFORE the append; the physical page of position ctx_len[b] must already be in
 *            page_table (pages are handed out by the caller)
 *   ctx_len_out  optional int32 [batch] = ctx_len + 1 (may be ctx_len itself)
 *   kv_new / kv_pool  optional HOST arrays of n_kv device pointers: row b of kv_new[i] ([batch, kv_row_bytes] bytes)
 *            is copied to the row of pool i that holds position ctx_len[b] (the attention caches of the group's
 *            layers); kv_row_bytes is a multiple of 16, n_kv <= 8; n_kv = 0 skips this.
 * One launch.  pooling = LSA_POOL_MINMAX returns LSA_ERR_SHAPE. */
LSA_API int lsa_append(lsa_ctx* ctx, const lsa_params* p, const void* k_new, void* k_idx, float* k_scale, void* kmean,
                       const int32_t* page_table, int64_t page_table_stride, const int32_t* ctx_len, int batch,
                       int32_t* ctx_len_out, int n_kv, const void* const* kv_new, void* const* kv_pool,
                       int64_t kv_row_bytes);

/* ---- a1-a4: the indexer (Eq. 9-12 with the scoring range of Eq. 7) -------------------------- */

/* For each query: eligible pages E = pages meeting C(t); if hi_enable and |E| > M keep the M pages
 * with the largest Eq.-9 score, else all of E; score the tokens of the kept pages inside C(t) with
 * Eq. 1 (fp32 accumulation of bf16 products; e4m3 keys are widened exactly and the per-token scale is
 * applied to the dot product); keep the Ksp largest.  With pooling = LSA_POOL_MINMAX the page score uses
 * s~ = sum_d max(q_d k_max_d, q_d k_min_d) (Eq. 13) in place of the mean-key dot product, computed as
 * [max(q,0) | min(q,0)] . [k_max | k_min]; `kmean` is then the extrema cache of lsa_block_means.
 *   q_idx       bf16 [n_query, H_I, d_I]       w  fp32 [n_query, H_I]
 *   k_idx/k_scale/kmean  as in lsa_block_means
 *   prefill (paged=0): query row i sits at position q_pos0+i; n_key tokens are cached (>= q_pos0+n_query);
 *                      page_table = ctx_len = NULL, batch = 1
 *   decode (paged=1):  n_query = batch; query b sits at ctx_len[b]-1; page_table int32
 *                      [batch, page_table_stride] maps logical page -> physical page
 *   sparse_idx  int32 [n_query, Ksp]  ascending positions (logical), padded with -1
 *   n_sparse    int32 [n_query]
 *   pages_out   optional int32 [n_query, M] kept pages ascending, -1 padded (NULL to skip)
 * Scratch: the page-score matrix fp32 [n_query, ceil(n_key_max/P)] in the workspace; for e4m3 caches with the
 * 64-head, 128-dim indexer also a bf16 copy of the codes [n_key_max, d_idx] (exact, unscaled), rewritten by every call,
 * from which the fine stage fetches key tiles. */
LSA_API int lsa_index(lsa_ctx* ctx, const lsa_params* p, const void* q_idx, const float* w, const void* k_idx,
              const float* k_scale, const void* kmean, int64_t q_pos0, int64_t n_query, int64_t n_key,
              const int32_t* page_table, int64_t page_table_stride, const int32_t* ctx_len, int batch,
              int32_t* sparse_idx, int32_t* n_sparse, int32_t* pages_out);

/* lsa_index for callers that can give the library no scratch memory.  (The paper has no counterpart:
 * this is a packaging variant of the prefill indexer above.)
 *
 * Who needs it: code that runs where device memory can no longer be obtained — inside a serving engine
 * that reserved the whole GPU for its own pools at start-up, from a plugin or callback that is handed
 * tensors but no allocator, or on a latency-critical path where an allocation (and the device-wide
 * synchronisation it may imply) is not acceptable.  Such callers cannot size and pass the workspace that
 * lsa_create / lsa_index expect.  Here the only scratch of the indexer, the page-score matrix
 * fp32 [n_query, ceil(n_key/P) rounded up to a multiple of 4], sits in a fixed array of
 * LSA_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads the library holds those bytes
 * until the process exits.  The call takes no lsa_ctx, allocates nothing on host or device and calls no
 * allocating routine.
 *
 * Kernels and results: the coarse stage is dispatched exactly as lsa_index dispatches it and the fine stage
 * is the same kernel, so sparse_idx / n_sparse are the ones lsa_index returns for the same inputs.  One
 * difference in speed: for e4m3 caches with the 64-head indexer lsa_index first writes a bf16 copy of the
 * codes into its workspace and feeds the fine stage from it by TMA; there is no room for that copy here, so
 * the fine stage gathers the codes and widens them in registers, which is slower.
 *
 * Arguments as lsa_index with paged = 0 (contiguous caches, query row i at position q_pos0+i) and the same
 * argument checks (LSA_ERR_SHAPE for a q_idx, w, k_idx or kmean that is not 16-byte aligned); `device` is the
 * CUDA device of all pointers, `cuda_stream` the stream to enqueue on.  No pages_out.  The caller's current
 * device is the same after the call as before it.
 * Limits and behaviour:
 *   - n_query * (ceil(n_key/P) rounded up to 4) * 4 bytes must not exceed LSA_STATIC_SCRATCH_BYTES, else
 *     LSA_ERR_CAPACITY and nothing is launched; split the queries over several calls.  Mean pooling,
 *     keep_pages * page <= 4096, and with hi_enable = 0 caches of at most 4096 tokens.
 *   - The first call on each device is a set-up call: it looks up the arrays' device addresses
 *     (cudaGetSymbolAddress, with that device made current), which is also when the CUDA runtime loads
 *     this part of the library onto the device — the array's bytes and the kernels' code are obtained from
 *     the driver then, not at dlopen.  Make that first call at start-up, before the application reserves
 *     the rest of the GPU's memory and before any stream capture begins; if the device has no room left
 *     it returns LSA_ERR_CUDA.
 *   - All calls on a device share the one array, which keeps the previous call's contents.  Nothing in it
 *     has to start at zero (the fine stage reads only entries the coarse stage of the same call wrote).
 *     Two calls whose kernels overlap on the GPU — different streams, or different host threads — race on
 *     it: order them on one stream or with events.
 *   - Device-side waits are bounded as everywhere in the library.  A wait that ran out leaves
 *     LSA_ERR_TIMEOUT in a status word that sits beside the array and is shared in the same way; read it
 *     with lsa_index_static_status. */
#define LSA_STATIC_SCRATCH_BYTES (8u << 20)
LSA_API int lsa_index_static(int device, void* cuda_stream, const lsa_params* p, const void* q_idx, const float* w,
                             const void* k_idx, const float* k_scale, const void* kmean, int64_t q_pos0,
                             int64_t n_query, int64_t n_key, int32_t* sparse_idx, int32_t* n_sparse);
/* Waits for `cuda_stream`, copies the status word of lsa_index_static on `device` to *device_status (0, or
 * LSA_ERR_TIMEOUT if a device-side wait of an earlier lsa_index_static call ran out, in which case that
 * call's outputs are not valid) and clears it.  Allocates nothing; the counterpart of lsa_status for the
 * entry point that has no context.  (No counterpart in the paper.) */
LSA_API int lsa_index_static_status(int device, void* cuda_stream, int* device_status);

/* The selection step alone (Eq. 2 / 7 / 10 / 12) on caller-given fp32 scores; bit-exact by definition.
 *   scores    fp32 [n_query, ld_scores], column c of row i is the score of candidate c
 *   cand_pos  NULL: candidate c is position c;  else int32 [n_query, n_cand] positions, -1 = absent
 *   apply_range 1: only positions inside C(q_pos0+i) (from k_sink, k_swa) take part; 0: all present
 *   idx_out   int32 [n_query, k] ascending positions, -1 padded;  n_out int32 [n_query]
 * n_cand is unlimited (scores are re-read from memory on every radix pass); k <= 8192. */
LSA_API int lsa_select(lsa_ctx* ctx, const lsa_params* p, const float* scores, int64_t ld_scores,
               const int32_t* cand_pos, int64_t q_pos0, int64_t n_query, int64_t n_cand, int32_t k,
               int32_t apply_range, int32_t* idx_out, int32_t* n_out);

/* ---- a5: streaming-aware conversion (Sec. 3.1) ---------------------------------------------- */

/* Lays the index set of each query out as cache rows in the order the attention kernel streams them:
 * [sink run | sparse rows ascending | window run].  In paged mode each position is translated to its
 * physical row  page_table[b][pos / kv_page] * kv_page + pos % kv_page, so that the sink and the window
 * become runs of whole contiguous pages and the R layers of the group share one translation.
 *   rows_out   int32 [n_query, k_sink + k_sparse + k_swa]   (-1 padded)     n_rows_out int32 [n_query]
 *   runs_out   optional int32 [n_query, 4] = {first sink row count, sparse count, window count,
 *              number of maximal runs of consecutive rows in the list}  (NULL to skip) */
LSA_API int lsa_convert(lsa_ctx* ctx, const lsa_params* p, const int32_t* sparse_idx, const int32_t* n_sparse,
                int64_t q_pos0, int64_t n_query, const int32_t* page_table, int64_t page_table_stride,
                const int32_t* ctx_len, int batch, int32_t* rows_out, int32_t* n_rows_out, int32_t* runs_out);

/* ---- a6: sparse attention (Eq. 3) ------------------------------------------------------------ */

/* out[t,h,:] = sum_{s in S_t} softmax_s(sm_scale * q[t,h].k[s]) * v[s,:d_v],  S_t = sink U window U sparse;
 * bf16 tensor-core products, fp32 softmax and accumulation; one softmax over the whole set.
 *   q    bf16 [n_query, H, d_qk]
 *   k    bf16 rows of ld_k elements (>= d_qk);  v bf16 rows of ld_v elements (>= d_v).  MLA latent: v == k.
 *   sparse_idx / n_sparse  as written by lsa_index (logical positions)
 *   rows / n_rows  optional output of lsa_convert; when given (required in paged mode) the kernel reads
 *                  these cache rows instead of rebuilding the set from sparse_idx
 *   out  bf16 [n_query, H, d_v]      lse  optional fp32 [n_query, H] = log sum_s exp(logit)
 * Paged mode splits each sequence's rows over several thread blocks; the partial results sit in the
 * workspace and are merged by their log-sum-exp. */
LSA_API int lsa_sparse_attn(lsa_ctx* ctx, const lsa_params* p, const void* q, const void* k, const void* v,
                    int64_t ld_k, int64_t ld_v, const int32_t* sparse_idx, const int32_t* n_sparse,
                    const int32_t* rows, const int32_t* n_rows, int64_t q_pos0, int64_t n_query,
                    int64_t n_key, const int32_t* ctx_len, int batch, void* out, float* lse);

/* Merge attention results over disjoint key sets by their log-sum-exp (the rescaling merge of the two-branch
 * operator, Sec. 4.1.1, and of the sharded-cache decode, App. B):
 *     lse = log sum_i exp(lse_i),   out = sum_i exp(lse_i - lse) * out_i.
 *   outs   HOST array of n_parts device pointers, each bf16 [n_query, H, d_v] (as written by lsa_sparse_attn)
 *   lses   HOST array of n_parts device pointers, each fp32 [n_query, H]; -inf marks an empty part
 *   out    bf16 [n_query, H, d_v]     lse  optional fp32 [n_query, H]
 * 1 <= n_parts <= 8.  A part is produced by lsa_sparse_attn with the budget of the other parts set to zero
 * (k_sparse = 0: sink + window only; k_sink = k_swa = 0: sparse only), or by a rank that holds a shard of the rows. */
LSA_API int lsa_merge(lsa_ctx* ctx, const lsa_params* p, int n_parts, const void* const* outs,
                      const float* const* lses, int64_t n_query, void* out, float* lse);

/* ---- a7: one cross-layer group (Sec. 3.2) ---------------------------------------------------- */

/* Indexer once (lsa_index, in passes of q_chunk queries when q_chunk > 0), conversion once, then the
 * attention of the R = n_layers layers one after the other on the context's stream, all with the same
 * index set.  q/k/v/out/lse are HOST arrays of R device pointers (lse or its entries may be NULL).
 * kmean must already hold the means (lsa_block_means) — the cache is maintained per sequence, not per
 * group.  sparse_idx / n_sparse are caller buffers, returned filled for inspection.
 * Paged mode: the conversion rides in the indexer's last kernel.  The layers are never launched side by side: in a
 * model the query of layer r + 1 is computed from the output of layer r. */
LSA_API int lsa_layer_group(lsa_ctx* ctx, const lsa_params* p, const void* q_idx, const float* w,
                    const void* k_idx, const float* k_scale, const void* kmean, int64_t q_pos0,
                    int64_t n_query, int64_t n_key, const int32_t* page_table, int64_t page_table_stride,
                    const int32_t* ctx_len, int batch, const void* const* q, const void* const* k,
                    const void* const* v, int64_t ld_k, int64_t ld_v, void* const* out, float* const* lse,
                    int32_t* sparse_idx, int32_t* n_sparse);

/* Same group, prefill only, with the per-query tensors in HOST memory (pinned for full speed):
 * q_idx_host, w_host, q_host[r], out_host[r] are host pointers (row i = the query at position q_pos0 + i); caches (k_idx, k_scale, kmean, k[r], v[r])
 * stay device-resident.  The queries are processed in passes of `stage_queries`; each pass copies its
 * slice of q_idx, w and q[r] to the device staging buffers, runs the group on it and copies out[r] back;
 * copies in, kernels and copies out of consecutive passes overlap on two internal streams (the copy-in of pass i+2
 * starts as soon as the kernels of pass i have read their inputs).
 * stage[2] are two caller-owned device staging areas of lsa_host_stage_bytes() bytes each. */
LSA_API int lsa_layer_group_host(lsa_ctx* ctx, const lsa_params* p, const void* q_idx_host, const float* w_host,
                         const void* k_idx, const float* k_scale, const void* kmean, int64_t q_pos0,
                         int64_t n_query, int64_t n_key, const void* const* q_host, const void* const* k,
                         const void* const* v, int64_t ld_k, int64_t ld_v, void* const* out_host,
                         int64_t stage_queries, void* const* stage, size_t stage_bytes);
LSA_API int lsa_host_stage_bytes(const lsa_params* p, int64_t stage_queries, size_t* bytes);

#ifdef __cplusplus
}
#endif
#endif /* LSA_H_ */
