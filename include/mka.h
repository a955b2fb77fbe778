/*
 * mka.h -- C ABI of the B200 (sm_100a) FastMKA attention library.
 *
 * The operator (paper, "Theoretical Formulation", Eq. 5): for every query token t a router gate
 * lambda_t in R^3 (non-negative, sums to one) weighs three memory levels -- L1 local window,
 * L2 session memory, L3 long-term slots -- and the output is the gated mixture of
 * exponentiated scores under ONE normalisation:
 *
 *     O_t = sum_l lambda_{t,l} sum_{j in vis_l(t)} exp(s_{t,l,j}) v_{l,j}  /  Z_t
 *     Z_t = sum_l lambda_{t,l} sum_{j in vis_l(t)} exp(s_{t,l,j}),   s_{t,l,j} = scale * q_t . k_{l,j}
 *
 * evaluated block-wise with a running maximum (Eq. 11-14; block partition Eq. 2-4, Alg. 3).
 * Visibility: with p = t + q_offset the position of query t on the key timeline,
 *     L1: j in (p - window, p]      (a causal window that ends at, and includes, the query's own row)
 *     L2: j in [0, p]               (causal prefix; one session entry per token)
 *     L3: j in [0, n_3)             (every recalled slot)
 * each intersected with [0, n_l).  A level with n_l = 0, or a row whose gate for that level is 0,
 * contributes nothing (Local-MKA = levels 1,2 only; "L1 only" = standard attention).
 *
 * General rules for every entry point
 *   - All data pointers are DEVICE pointers unless a parameter says "host".  Structs (mka_shape,
 *     mka_level[3], ...) are read on the host during the call.
 *   - The caller owns every buffer; the library allocates no device memory and keeps no state
 *     between calls.  Scratch memory comes from the caller as `ws` (size from mka_workspace_bytes).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls only enqueue work;
 *     they do not synchronise.  Outputs are fully overwritten.
 *   - Errors are reported by return code only; arguments are validated on the host before anything
 *     is launched, and nothing is launched when validation fails.  No entry point aborts or traps.
 *   - Head width d must be 32, 64, 96 or 128 (decode and the tensor-core forward: 64 or 128).  bf16 tensors
 *     need 16-byte aligned base pointers and strides that are multiples of 8 elements.
 *   - There is no CPU fallback: without a CUDA device every compute entry point returns MKA_ERR_CUDA.
 */
#ifndef MKA_H_
#define MKA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MKA_OK = 0,
    MKA_ERR_ARG = 1,          /* null pointer, bad enum value */
    MKA_ERR_SHAPE = 2,        /* non-positive size, unsupported head width, window < 1 */
    MKA_ERR_ALIGN = 3,        /* pointer or stride alignment */
    MKA_ERR_WORKSPACE = 4,    /* ws == NULL or ws_bytes too small */
    MKA_ERR_UNSUPPORTED = 5,  /* combination not implemented (e.g. MKA_MODE_FULL backward) */
    MKA_ERR_CUDA = 6,         /* a CUDA runtime call failed (no device, launch failure) */
    MKA_ERR_TIMEOUT = 7       /* a bounded device-side wait expired (see mka_device_status) */
} mka_status;

typedef enum { MKA_BF16 = 0, MKA_F32 = 1 } mka_dtype;

/* MKA_MODE_FAST: Eq. 5 (FastMKA: one attention pass, one normalisation).
 * MKA_MODE_FULL: Alg. 1 (Symbolic MKA): one softmax attention per level, outputs mixed by the gate. */
typedef enum { MKA_MODE_FAST = 0, MKA_MODE_FULL = 1 } mka_mode;

/* Routing variants of the gate (Alg. 1 "lambda <- softmax(MLP(q))"; hard top-k and fixed 1/3 are the
 * routing-ablation variants of Table 10). */
typedef enum { MKA_ROUTE_SOFT = 0, MKA_ROUTE_UNIFORM = 1, MKA_ROUTE_TOP1 = 2, MKA_ROUTE_TOP2 = 3 } mka_route;

/* mka_shape.flags */
#define MKA_FLAG_FORCE_SIMT 1u   /* run the CUDA-core kernels even where a tensor-core kernel exists */
#define MKA_FLAG_TEST_STALL 0x80000000u /* test hook of mka_fwd (tensor-core kernel, dense levels): the loader of every
                                           CTA leaves out its last key tile, so the wait for that tile runs into the
                                           limit of mka_set_wait_limit_us and the call ends with MKA_ERR_TIMEOUT in
                                           the status word; O and LSE of such a call are invalid.  In mka_bwd
                                           (tensor-core kernels) the loader of every CTA of the dK/dV kernel leaves
                                           out its last query tile, with the same end; the gradients of such a call
                                           are invalid.  Exists so that the give-up path can be exercised without a
                                           fault or a hang. */

/* which = argument of mka_workspace_bytes */
#define MKA_WS_FWD 0
#define MKA_WS_DECODE 1
#define MKA_WS_BWD 2

/* One memory level's key/value source: k, v are [B, H, n, d] with d contiguous and explicit strides
 * (in ELEMENTS) for the batch, head and row dimensions.  n may be 0 (then k, v may be NULL). */
typedef struct mka_level {
    const void *k, *v;
    int64_t n;
    int64_t stride_b, stride_h, stride_n;
} mka_level;

/* Gradient destinations for one level, same geometry as mka_level. */
typedef struct mka_level_grad {
    void *dk, *dv;
    int64_t n;
    int64_t stride_b, stride_h, stride_n;
} mka_level_grad;

/* Problem shape in the paper's notation: B batch, H heads, T query tokens, d head width, D model
 * width (router input width); window = W of the L1 level; q_offset = key-timeline position of query 0;
 * scale = tau of Eq. 3 (<= 0 selects 1/sqrt(d)). */
typedef struct mka_shape {
    int32_t B, H, T, d, D;
    int32_t window;
    int32_t q_offset;
    float scale;
    int32_t dtype;   /* mka_dtype of Q, K, V, O, dO, dQ, dK, dV */
    int32_t mode;    /* mka_mode */
    uint32_t flags;  /* MKA_FLAG_* */
    int32_t kv_heads; /* grouped-query sharing (the paper evaluates on GQA models): 0 or H = one KV head per query
                         head; otherwise H % kv_heads == 0, the levels hold kv_heads heads ([B, kv_heads, n, d]) and
                         query head h reads KV head h / (H / kv_heads).  Honoured by mka_fwd, mka_decode and
                         mka_bwd (dK, dV then hold kv_heads heads, summed over each group); the paged entry points
                         take H_kv as an argument instead */
} mka_shape;

/* Split table of the decode kernel: level l is cut into n_chunks[l] chunks of chunk_rows rows (the last
 * one shorter); chunk c of level l covers rows [c*chunk_rows, min(n_l, (c+1)*chunk_rows)). */
typedef struct mka_decode_plan_t {
    int64_t chunk_rows;
    int64_t n_chunks[3];
    int64_t total_chunks;   /* per (batch, head) */
} mka_decode_plan_t;

/* Key-tile range of one 128-row query tile on one level, in units of 128-row key tiles:
 * tiles [first, end) hold at least one visible pair; tiles [full_first, full_end) within it are
 * visible to every row of the query tile and need no element mask. */
typedef struct mka_tile_range {
    int64_t first, end, full_first, full_end;
} mka_tile_range;

const char* mka_status_str(mka_status s);

/*
 * Router gate (Alg. 1 step 12 / Alg. 2 step 5, read as one linear layer followed by a softmax over
 * the three levels; one gate per token, shared by all heads).
 *   R        [rows, D] router input, row-major, r_dtype (bf16 or f32)
 *   W_r      [D, 3] f32, b_r [3] f32 or NULL (zero bias)
 *   route    MKA_ROUTE_*: SOFT = softmax; UNIFORM = 1/3 each; TOP1/TOP2 = keep the 1/2 largest logits
 *            (ties go to the lower level index), renormalise the kept gates, others exactly 0
 *   gate     [rows, 3] f32 out
 *   log2_gate[rows, 3] f32 out or NULL: log2 of the gate (-inf where the gate is 0)
 *   route_idx[rows, 2] int8 out or NULL: kept level indices ascending, -1 = unused slot
 *            (both -1 for SOFT and UNIFORM)
 * rows == 0 is valid and launches nothing.
 */
mka_status mka_router(const void* R, const float* W_r, const float* b_r, int64_t rows, int32_t D,
                      int32_t r_dtype, int32_t route, float* gate, float* log2_gate, int8_t* route_idx,
                      void* stream);

/* Bytes of caller-provided scratch the given entry point needs (host function, no CUDA call).
 * n_level = rows of the three levels.  Returns 0 on invalid arguments. */
size_t mka_workspace_bytes(const mka_shape* shape, const int64_t n_level[3], int32_t which);

/*
 * Fused forward (Eq. 5 block-wise with the running maximum of Eq. 11-14; MKA_MODE_FULL: Alg. 1).
 *   Q    [B, H, T, d] contiguous;  L[3] level sources;  gate [B, T, 3] f32 (an INPUT: >= 0)
 *   O    [B, H, T, d] out, same dtype as Q (rounded once, to nearest even, for bf16)
 *   LSE  [B, H, T] f32 out or NULL: natural log of Z_t (-inf and O = 0 where nothing is visible);
 *        not written in MKA_MODE_FULL
 * bf16 with d in {64,128} runs the TMA + tcgen05 kernel; f32, MKA_MODE_FULL and MKA_FLAG_FORCE_SIMT
 * run the CUDA-core kernel.
 */
mka_status mka_fwd(const mka_shape* shape, const void* Q, const mka_level L[3], const float* gate,
                   void* O, float* LSE, void* ws, size_t ws_bytes, void* stream);

/*
 * Split-KV single-token decode: Eq. 5 for T == 1 where EVERY cached row of every level is visible
 * (window and q_offset are ignored).  Each chunk of the split table produces an un-gated partial
 * (max, sum, accumulator); a second kernel combines them with the gate in log-sum-exp form.
 *   q [B, H, d];  gate [B, 3] f32;  O [B, H, d];  LSE [B, H] f32 or NULL.
 * With shape->kv_heads < H (at most 16 query heads per KV head) the grouped-query kernel of mka_decode_paged runs on the
 * dense levels and reads every cached row once per KV head; ask mka_workspace_bytes with the same shape.
 */
mka_status mka_decode(const mka_shape* shape, const void* q, const mka_level L[3], const float* gate,
                      void* O, float* LSE, void* ws, size_t ws_bytes, void* stream);

/* One memory level kept in PAGES (the paged KV layout the paper's inference setup uses for contexts beyond 32K):
 * pools k, v hold fixed-size pages; element (page, kv head, row, :) sits at page*stride_page + head*stride_h +
 * row*stride_n (ELEMENTS, d contiguous).  Logical row r of sequence b is row r % page_rows of pool page
 * page_table[b*table_stride + h*table_head_stride + r / page_rows].  n may be 0 (then the pointers may be NULL). */
typedef struct mka_paged_level {
    const void *k, *v;          /* device, bf16 */
    const int32_t* page_table;  /* device [B, table_stride]; entries of pages that hold no valid row are never read */
    const int32_t* rows;        /* device [B]: valid rows of every sequence (clamped to [0, n]), or NULL = n for all */
    int64_t n;                  /* upper bound of the sequences' rows (host); table_stride * page_rows >= n */
    int64_t table_stride;
    int64_t table_head_stride;  /* 0 = one table per sequence; else KV head h of sequence b uses the table at
                                   b*table_stride + h*table_head_stride (per-head recall lists of mka_l3_retrieve) */
    int32_t page_rows;          /* rows per page: a power of two */
    int64_t stride_page, stride_h, stride_n;
    int64_t pool_pages;         /* pages in the pool; read by mka_fwd_paged only (mka_decode_paged ignores it) */
} mka_paged_level;

/*
 * Split-KV single-token decode over paged levels with grouped-query sharing of the KV heads (the paper evaluates on
 * GQA models and serves long contexts from a paged KV cache; Eq. 5 itself is unchanged): same result as mka_decode on
 * the gathered, head-repeated levels.  shape->H query heads share H_kv KV heads, consecutive query heads one KV head
 * (head h reads KV head h / (H / H_kv)); H must be a multiple of H_kv with at most 16 query heads per KV head.
 * Every cached row is read once per KV head.  A level whose gate is exactly 0 for a sequence is not read.
 *   q [B, H, d] bf16;  gate [B, 3] f32;  O [B, H, d] bf16;  LSE [B, H] f32 or NULL
 *   ws: mka_decode_paged_workspace_bytes(shape, H_kv, n_level) bytes, n_level[l] = L[l].n.  The levels are split into
 *       chunks of a multiple of 128 rows (at most 8192), chosen so that the grid makes few rounds of the resident CTAs
 * d must be 64 or 128; pools 16-byte aligned with strides that are multiples of 8 elements.
 * Levels whose pages hold at least 8 rows (and dense levels, see mka_decode) are streamed by the copy engine: a
 * producing warp issues one tensor-map copy per page and 64-column panel, the computing warps wait on barriers for
 * them.  Those waits are bounded (mka_set_wait_limit_us; mka_device_status(ws) then reads MKA_ERR_TIMEOUT).  Rows of a
 * partly filled page after a sequence's last row may hold anything, NaN included; pages without a valid row are never read.
 */
size_t mka_decode_paged_workspace_bytes(const mka_shape* shape, int32_t H_kv, const int64_t n_level[3]);
mka_status mka_decode_paged(const mka_shape* shape, int32_t H_kv, const void* q, const mka_paged_level L[3],
                            const float* gate, void* O, float* LSE, void* ws, size_t ws_bytes, void* stream);

/*
 * Fused forward of mka_fwd over paged levels (prefill, or a chunk of it, against a paged KV cache) with grouped-query
 * sharing: same result as mka_fwd on the gathered levels with shape->kv_heads = H_kv.  Sequence b has rows[b] rows on
 * level l (L[l].n for all when rows is NULL); all sequences share T and q_offset.  page_rows must be a power of two
 * >= 8; pool_pages must be set.  Rows of a sequence's last page after its last row may hold anything (NaN and Inf
 * included): the page is copied whole, the key rows are masked and the value rows are cleared in shared memory before
 * the product reads them.  Pages with no valid row are never read.
 * bf16, MKA_MODE_FAST, d in {64, 128} only (the TMA + tcgen05 kernel; a 128-row key tile is assembled from one box
 * per page); anything else returns MKA_ERR_UNSUPPORTED.  ws: at least 256 bytes (status word).
 */
mka_status mka_fwd_paged(const mka_shape* shape, int32_t H_kv, const void* Q, const mka_paged_level L[3],
                         const float* gate, void* O, float* LSE, void* ws, size_t ws_bytes, void* stream);

/*
 * L3 recall (Alg. 2 step 4 "L3 <- Retrieve(Q_h)"; the method section's vectorized hashing with chunk-based recall; the
 * passkey table recalls R = 8 chunks per query).  The paper does not define the hash; this library's reading: a chunk
 * is one page of the long-term key pool, its signature a sign-random-projection code of the SUM of its keys
 * (bit j = [proj[j] . sum >= 0]); the query of a KV head is the sum of the query heads that share it; the R chunks of
 * the sequence's bank whose codes agree with the query's code in the most bits are recalled, ties to the earlier
 * chunk, and listed in bank (time) order.  Code bits are decided in fp32: sums run row by row (head by head for the
 * query), a projection is one fmaf chain over the columns 0..d-1.
 *
 * mka_l3_index: codes of every (page, KV head) of a key pool.
 *   k_pool   bf16 pool, element (page, head, row, :) at page*stride_page + head*stride_h + row*stride_n; all
 *            page_rows rows of a page are summed (unused rows of a partly filled page must be zero)
 *   proj     [bits, d] f32, bits in {32, 64, 128, 256}; d in {64, 128}
 *   codes    [n_pages, H_kv, bits/32] uint32 out: bit j of a code is bit j%32 of word j/32
 * mka_l3_retrieve: per (sequence, KV head) the page table of the recalled chunks.
 *   q        [B, H, d] bf16;  codes from mka_l3_index with the same proj
 *   bank     int32 [B, bank_stride]: pool pages of each sequence's long-term chunks in time order; bank_len int32 [B]
 *            how many are in use (clamped to [0, max_bank]); max_bank (host) <= bank_stride, at most 98304 (the scores of a bank live in shared memory)
 *   R        chunks to recall, 1..64
 *   table    int32 [B, H_kv, R] out: recalled pool pages in bank order, unused slots 0
 *   n_sel    int32 [B] out or NULL: min(R, bank_len[b]);  rows int32 [B] out or NULL: n_sel * page_rows
 * The outputs plug into mka_paged_level (page_table = table, table_stride = H_kv*R, table_head_stride = R, rows).
 */
mka_status mka_l3_index(const void* k_pool, int64_t n_pages, int32_t H_kv, int32_t page_rows, int32_t d,
                        int64_t stride_page, int64_t stride_h, int64_t stride_n, const float* proj, int32_t bits,
                        uint32_t* codes, void* stream);
mka_status mka_l3_retrieve(const void* q, int32_t B, int32_t H, int32_t H_kv, int32_t d, const float* proj,
                           int32_t bits, const uint32_t* codes, const int32_t* bank, const int32_t* bank_len,
                           int64_t bank_stride, int32_t max_bank, int32_t R, int32_t page_rows, int32_t* table,
                           int32_t* n_sel, int32_t* rows, void* stream);

/*
 * Backward of mka_fwd in MKA_MODE_FAST (derived from Eq. 5; the paper prints no backward).  With
 * p = lambda exp(s - LSE) on the visible set and D_t = dO_t . O_t:
 *   dV = p^T dO,  dS = p (dO v^T - D),  dQ = scale dS K,  dK = scale dS^T Q,
 *   dG[b,t,l] = sum over heads and visible j of dS   (gradient w.r.t. the router LOGIT of level l),
 *   dW_r = R^T dG,  db_r = sum dG.
 *   O, LSE: outputs of mka_fwd;  dO [B,H,T,d];  R [B*T, D] router input in r_dtype (NULL skips dW_r, db_r)
 *   dQ [B,H,T,d];  dL[3] gradient destinations (a level with n == 0 is skipped);  dG [B,T,3] f32;
 *   dW_r [D,3] f32 or NULL;  db_r [3] f32 or NULL.
 * dG is the logit gradient of a gate that is a softmax of the logits (MKA_ROUTE_SOFT; for TOP1 / TOP2 the renormalised
 * softmax over the kept levels, whose dropped levels get dG = 0 because their gate is 0).  dW_r = R^T dG and
 * db_r = sum dG follow from that; with MKA_ROUTE_UNIFORM the gate does not depend on W_r, so the true dW_r, db_r are 0
 * and a caller training that variant passes dW_r = db_r = NULL.
 * bf16 with d in {64,128} runs the TMA + tcgen05 kernels (one pass that owns query tiles for dQ and dG, one
 * pass that owns key tiles for dK and dV; scores are recomputed in each, nothing is accumulated atomically);
 * f32, other head widths and MKA_FLAG_FORCE_SIMT run the CUDA-core kernels.  Both are deterministic.
 */
mka_status mka_bwd(const mka_shape* shape, const void* Q, const mka_level L[3], const float* gate,
                   const void* O, const float* LSE, const void* dO, const void* R, int32_t r_dtype,
                   void* dQ, const mka_level_grad dL[3], float* dG, float* dW_r, float* db_r,
                   void* ws, size_t ws_bytes, void* stream);

/*
 * Route-fusion with cache write (Alg. 2 steps 6-8).  Alg. 2 mixes the three token-aligned level representations of
 * every token with that token's own gate BEFORE the key/value projection and appends the projected result to ONE
 * cache; because the projection is linear the same cache rows are obtained by mixing the projected levels:
 *     dst.dk[b,h,dst_offset + j,:] = sum_l gate[b,j,l] * L[l].k[b,h,j,:]     (and likewise dv from L[l].v)
 * for j in [0, n).  Attention over that single cache is then mka_fwd / mka_decode with one level.
 *   B, H, n, d   sizes; d a multiple of 8 (bf16) or 4 (f32), at most 1024; H = 1 and d = D fuses the level
 *                representations [B, n, D] themselves (step 6 taken literally)
 *   L[3]         level sources; each L[l].n must be n, or 0 for an absent level (its gate is then ignored);
 *                a gate that is exactly 0 drops its level's values whatever they are
 *   gate         [B, n, 3] f32: the gate of the token the row belongs to
 *   dst          destinations: dk, dv with their strides; dst->n = rows of the destination (capacity);
 *                rows [dst_offset, dst_offset + n) are written, nothing else is touched
 * fp32 accumulation, one rounding to the storage type.  16-byte alignment rules as for the other entry points.
 */
mka_status mka_fuse_kv(int32_t B, int32_t H, int64_t n, int32_t d, int32_t dtype, const mka_level L[3],
                       const float* gate, const mka_level_grad* dst, int64_t dst_offset, void* stream);

/*
 * mka_fuse_kv with a PAGED destination: the fused rows of sequence b are appended to a paged cache at logical rows
 * dst_offset + dst_offsets[b] + j (dst_offsets: device int32 [B], or NULL = 0 for all), found through dst->page_table
 * as in mka_paged_level (one table per sequence; table_head_stride is ignored).  dst->k, dst->v are WRITTEN although
 * the struct declares them const; H counts the heads of the pool.  dst->n and the table must cover dst_offset + n rows
 * plus the largest per-sequence offset (the latter is the caller's promise: it lives on the device).  Everything else
 * as mka_fuse_kv.
 */
mka_status mka_fuse_kv_paged(int32_t B, int32_t H, int64_t n, int32_t d, int32_t dtype, const mka_level L[3],
                             const float* gate, const mka_paged_level* dst, int64_t dst_offset, const int32_t* dst_offsets,
                             void* stream);

/* Causal summaries of mka_l2_summary. */
typedef enum { MKA_SUMMARY_MEAN = 0, MKA_SUMMARY_EMA = 1 } mka_summary;
/* Test hook, OR-ed into `kind` (segmented form only): segment 1 of every column strip never publishes its carried
 * state, so the look-back of the later segments runs into the limit of mka_set_wait_limit_us and the call ends with
 * MKA_ERR_TIMEOUT in the status word; M2 and state of such a call are invalid. */
#define MKA_SUMMARY_TEST_STALL 0x40000000

/*
 * L2 session summary (Alg. 1, the loop "M_2[t] <- Summary(X[:, 1:t, :])", named there as "prefix mean or EMA";
 * Alg. 2 step 3): a causal scan along the sequence that produces the L2 level's source.  Row t of M2 summarises
 * rows 0..t of X and nothing later:
 *   MKA_SUMMARY_MEAN   M2[b,t,:] = (S + sum_{i<=t} X[b,i,:]) / (n_prev + t + 1)
 *   MKA_SUMMARY_EMA    m_t = beta m_{t-1} + (1 - beta) X[b,t,:],  M2[b,t,:] = m_t;  a fresh session starts with m_0 = X[b,0,:]
 *   X, M2   [B, T, D] contiguous, same dtype (bf16 or f32); D a multiple of 8 (bf16) / 4 (f32); 16-byte aligned
 *   state   [B, D] f32 or NULL.  With n_prev > 0 it is READ as the session's carried state (MEAN: the running sum S of
 *           the n_prev earlier tokens; EMA: m_{-1}); with n_prev == 0 the session is fresh and it is ignored on entry.
 *           When not NULL it is WRITTEN with the state to carry into the session's next chunk.
 *   beta    EMA decay in [0, 1]; ignored for MEAN
 *   ws      optional scratch.  With at least 256 bytes its first word receives the device status (mka_device_status).
 *           With mka_l2_summary_workspace_bytes(B, T, D, dtype) bytes (and ws 16-byte aligned) the sequences are cut
 *           into 256-row segments whose carried states are chained through the scratch, which keeps the whole GPU
 *           busy even for one long sequence; without it one CTA walks each strip of columns from end to end.  Both forms
 *           are single-pass and give the same results up to fp32 summation order.  NULL = no scratch, no status word.
 * fp32 arithmetic, one rounding to the storage type.  Counts are converted to f32 (exact up to 2^24 tokens).
 */
mka_status mka_l2_summary(const void* X, int32_t B, int64_t T, int32_t D, int32_t dtype, int32_t kind, float beta,
                          float* state, int64_t n_prev, void* M2, void* ws, size_t ws_bytes, void* stream);
/* Scratch bytes that let mka_l2_summary use its segmented form: 512 + 8 bytes per segment and column (about 1.6 % of
 * a bf16 input).  The call clears the scratch on its stream, so its contents on entry do not matter.  Host only. */
size_t mka_l2_summary_workspace_bytes(int32_t B, int64_t T, int32_t D, int32_t dtype);
/* 1 when mka_l2_summary would run the segmented form for this input with ws_bytes of scratch (T >= 512, enough
 * scratch, and for fp32 fewer than 96 strips of 128 bytes over all sequences), else 0 (the strip form).  Host only. */
int32_t mka_l2_summary_kernel_kind(int32_t B, int64_t T, int32_t D, int32_t dtype, size_t ws_bytes);


/*
 * Decode for callers that cannot provide scratch memory (the paper has no counterpart; this entry
 * point exists for deployment reasons only).  Same computation, arguments and results as mka_decode,
 * but without `ws`: the per-chunk partials are kept in an 8 MiB array that is compiled into the
 * library, so the call performs no device allocation of any kind and needs none from its caller.
 * It is meant for hosts where allocating is not an option at call time: serving engines that claim
 * all device memory for their own pool at start-up (a later cudaMalloc there fails or has to wait for
 * the device to go idle), latency-bound decode loops that may not stall on the allocator's implicit
 * device synchronisation, and plug-ins that only ever receive raw input/output pointers from a
 * runtime whose memory plan is fixed before the first token.
 *   - Limit: B * H * total_chunks * (d + 2) floats (total_chunks from mka_decode_plan) must fit in
 *     mka_decode_static_max_bytes() = 8 MiB; larger problems are rejected with MKA_ERR_WORKSPACE and
 *     nothing is launched.  (For d = 128 that is 16131 chunk partials, e.g. 32 heads x 516k cached rows.)
 *   - The array costs 8 MiB on every GPU that runs a decode kernel of this library, for the life of the
 *     process.  The CUDA runtime sets it aside when this part of the library is first used on a device (the
 *     first decode call, or the address look-up below), not when the library is loaded; on a device whose
 *     memory is already exhausted that first use fails and the call returns MKA_ERR_CUDA.
 *   - The first call on each device looks up the array's device address (with that device current)
 *     and remembers it; make that first call during set-up, before any stream capture begins.  The
 *     remembered address does not survive a cudaDeviceReset of that device.
 *   - All calls on one device share the one array and it keeps whatever the last call wrote.  Nothing
 *     in it needs clearing between calls (every slot that is read was written by the same call), but
 *     two calls whose kernels overlap on the GPU -- different streams, no ordering between them --
 *     race on it and produce garbage.  Serialise such calls or use mka_decode with separate workspaces.
 */
mka_status mka_decode_static(const mka_shape* shape, const void* q, const mka_level L[3], const float* gate,
                             void* O, float* LSE, void* stream);
size_t mka_decode_static_max_bytes(void);

/* Integer bookkeeping, exposed so that it can be checked bit for bit (host functions, no CUDA call). */
mka_status mka_decode_plan(const int64_t n_level[3], int32_t B, int32_t H, int32_t d, mka_decode_plan_t* plan);
mka_status mka_fwd_tile_range(const mka_shape* shape, const int64_t n_level[3], int32_t level,
                              int64_t q_tile, mka_tile_range* out);

/* Which forward kernel mka_fwd would run for this problem (host function, no launch):
 * 0 = CUDA-core kernel, 1 = TMA + tcgen05 tensor-core kernel, negative = arguments invalid. */
int32_t mka_fwd_kernel_kind(const mka_shape* shape, const mka_level L[3]);

/* Which kernels mka_bwd would run for this problem (host function, no launch): 0 = CUDA-core kernels,
 * 1 = TMA + tcgen05 tensor-core kernels (bf16, d in {64,128}, 16-byte aligned strides), negative = arguments
 * invalid.  dL may be NULL (then only the level sources decide). */
int32_t mka_bwd_kernel_kind(const mka_shape* shape, const mka_level L[3], const mka_level_grad dL[3]);

/* Synchronises `stream` and returns the device status word that the kernels of the last call using
 * `ws` left there: MKA_OK, or MKA_ERR_TIMEOUT when a bounded wait inside a kernel gave up (the
 * kernel then released its resources and returned; outputs of that call are invalid). */
mka_status mka_device_status(const void* ws, void* stream);

/* Limit, in microseconds, of every wait inside the kernels (a warp waiting for a tile to land, for another warp's
 * result, for an earlier segment's state).  A wait that reaches it gives up: the CTA releases what it holds, the kernel
 * returns and the status word of the call's workspace reads MKA_ERR_TIMEOUT.  Default 1 000 000 (one second, far above
 * anything a healthy launch needs); 0 restores the default; values are clamped to [100, 10 000 000].  Process-wide,
 * read when a call is made.  Returns the previous value.  Host function, no CUDA call. */
uint32_t mka_set_wait_limit_us(uint32_t us);

#ifdef __cplusplus
}
#endif
#endif /* MKA_H_ */
