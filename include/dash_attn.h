/*
 * dash_attn.h -- C ABI of the DashAttention forward pass for NVIDIA B200 (sm_100a).
 *
 * The forward pass has three stages (paper Section 3):
 *   Stage 0  chunk summaries          kbar_c = softmax(<qbar, k_t>/sqrt(d))-weighted mean of the B keys
 *                                     of chunk c                                   (Eq. 3, Algorithm 1)
 *   Stage 1  alpha-entmax routing     x = gamma (alpha-1) <q, kbar_c>/sqrt(d) over the chunks before the
 *                                     query's own; per head tau with sum [x-tau]_+^(1/(alpha-1)) = 1;
 *                                     group weight w = mean over the GQA group; support = {w > 0};
 *                                     bias d_c = (log w_c - mean log w)/sigma
 *                                                         (Eq. 2, Eq. 4, Algorithm 2, Proposition 1)
 *   Stage 2  softmax attention over the tokens of the routed chunks plus the causal part of the
 *            query's own chunk, logits <q,k>/sqrt(d) + d_c (0 on the own chunk)
 *                                                         (Eq. 7, Proposition 1, Algorithm 3)
 *
 * Conventions
 *   - Every pointer is DEVICE memory unless its comment says "host".  The caller owns every buffer;
 *     the library allocates nothing, launches only on `stream` and keeps no state that affects results
 *     (what it does keep, per process: a launch counter, per-device caches of the SM count, of the
 *     architecture check and of which kernels had their shared-memory limit raised, and the fixed scratch
 *     array of dash_attn_attend_decode_static).
 *   - Calls are asynchronous: they return after enqueueing.  Argument errors are detected on the host
 *     before anything is enqueued and are returned synchronously.  Problems only a kernel can see
 *     (a bounded wait that ran out, a capacity overrun) are written to a status word at the start of
 *     the workspace; dash_attn_last_status() synchronises the stream and returns it.
 *   - Tensors are strided: stride arrays give element strides of (batch, token, head); the head_dim
 *     axis is contiguous.  Base pointers must be 16-byte aligned, strides multiples of 8 elements.
 *   - 0-based positions.  Chunk of token j is j / block.  T_s = seq_kv / block complete chunks have
 *     summaries; T_a = ceil(seq_kv / block) chunks exist; W = ceil(T_a / 32) mask words per row.
 *   - Query head h uses KV head h / (h_q / h_kv) (Section 3.2).
 *   - Which kernels run: bf16 tensors take the TMA / tcgen05 kernels (head_dim 64 or 128, every chunk size; prefill
 *     needs g_q = h_q / h_kv >= 2, decode takes every group size); fp32 tensors, g_q = 1 in prefill and the
 *     non-causal mode take CUDA-core kernels that compute the same thing (the correctness path).
 *     The choice is made from the parameters alone, never from the data, and is the same on every call.
 *   - causal = 1 is the paper's setting and the one the tensor-core kernels serve.  causal = 0 (prefill only;
 *     the paper does not define it) is read as: every complete chunk is a candidate of every row; the
 *     incomplete tail chunk (index T_s, present when seq_kv is not a multiple of block) takes the own chunk's
 *     part -- attended whole by every row with bias 0 -- and there is no causal mask.  It runs on the CUDA-core
 *     kernels; the list region of row i then starts at (b*h_kv + r) * seq_q * T_s + i * T_s.  A decode shape
 *     with causal = 0 returns DASH_ERR_UNSUPPORTED, causal = 0 with local_blocks > 0 DASH_ERR_INVALID_ARG.
 *   - Local window (p->local_blocks = L > 0): the chunks c_own-L .. c_own-1 of a row are not candidates of
 *     the entmax routing; they are attended like the own chunk (all their tokens, bias 0) and do not enter
 *     the mean of log w.  In the routing outputs they appear as ordinary list entries with bias exactly 0
 *     behind the routed ones (they have the largest chunk indices), their mask bits are set and count
 *     includes them, so Stage 2 needs no other description of the window.
 *
 * Routing outputs (Stage 1 -> Stage 2)
 *   mask     uint32 [batch, h_kv, seq_q, W]: bit (c & 31) of word (c >> 5) is set iff chunk c is
 *            attended by that row: the routed chunks and the row's own chunk (Algorithm 2, last step).
 *   count    int32 [batch, h_kv, seq_q]: number of routed chunks (own chunk not counted).
 *   blk_idx, blk_bias   compact per-row lists, ascending chunk index, own chunk excluded.  The list of
 *            row (b, r, i) starts at entry dash_attn_list_offset(p, b, r, i) and holds count entries;
 *            its region has room for every candidate chunk of the row, so regions never overlap:
 *              prefill: offset = (b*h_kv + r) * R + block*c*(c-1)/2 + (i % block)*c,  c = i / block,
 *                       with the candidate count of a row in the incomplete tail chunk clamped to T_s,
 *                       R = sum over rows of their candidate counts;
 *              decode : offset = (b*h_kv + r) * T_s.
 */
#ifndef DASH_ATTN_H_
#define DASH_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DASH_OK = 0,
  DASH_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, bad stride/alignment, struct_size mismatch */
  DASH_ERR_UNSUPPORTED = -2, /* valid request outside what is built (head_dim, block, non-causal decode, ...) */
  DASH_ERR_WORKSPACE = -3,   /* workspace null, misaligned or smaller than dash_attn_workspace_bytes() */
  DASH_ERR_CAPACITY = -4,    /* device side: a list or queue overran its region */
  DASH_ERR_CUDA = -5,        /* a CUDA runtime / driver call failed */
  DASH_ERR_ARCH = -6,        /* the current device is not compute capability 10.x */
  DASH_ERR_TIMEOUT = -7,     /* device side: a bounded wait (mbarrier) ran out; results are invalid */
  DASH_ERR_TOO_LARGE = -8    /* the problem needs more scratch than a *_static entry point's fixed array holds */
} dash_status;

typedef enum { DASH_F32 = 0, DASH_BF16 = 1 } dash_dtype;

/* Problem statement (Section 3, "Problem setup and notation"; Algorithms 1-3 inputs). */
typedef struct dash_params {
  uint32_t struct_size; /* sizeof(dash_params); checked */
  int32_t batch;
  int32_t seq_q;        /* prefill: n (must equal seq_kv); decode: 1 */
  int32_t seq_kv;       /* prefill: n; decode: capacity of the KV cache in tokens */
  int32_t h_q, h_kv;    /* h_q % h_kv == 0 */
  int32_t head_dim;     /* 64 or 128 */
  int32_t block;        /* chunk size B: 16, 32, 64 or 128 */
  int32_t dtype;        /* dash_dtype of Q, K, V, O */
  int32_t causal;       /* 1 (the paper's setting) or 0 (see Conventions) */
  float alpha;          /* > 1; 1.25, 1.5 and 2 have integer exponents and take the fast path */
  float gamma;          /* Stage-1 temperature multiplying the chunk logit (Eq. 4) */
  float sigma;          /* prior strength of Eq. 8, > 0 */
  int32_t local_blocks; /* L >= 0 window chunks before the own chunk that every row attends in full with
                           bias 0 and that are not scored (appendix "Long-context adaptation": the sliding
                           window of the trained models is the own chunk plus the previous one, L = 1);
                           0 = Algorithms 2-3 as printed */
  const int32_t* q_to_kv; /* host, h_q entries, or NULL for h / (h_q/h_kv); only that map is accepted */
  int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3]; /* elements: batch, token, head */
} dash_params;

/* Bytes of workspace that select / fwd_prefill / fwd_decode / attend_* need for these parameters
 * (0 if the parameters are invalid).  The workspace must be 256-byte aligned.  It starts with the
 * status word followed by arrival counters that the library keeps at zero between calls (16,640 bytes
 * in all, cleared by dash_attn_reset_status, which must therefore run once before the first use);
 * the rest is scratch whose contents mean nothing between calls. */
size_t dash_attn_workspace_bytes(const dash_params* p);

/* Entries the blk_idx / blk_bias lists need, and where a row's region starts (see top of file).
 * Both return -1 for invalid parameters or indices. */
int64_t dash_attn_list_capacity(const dash_params* p);
int64_t dash_attn_list_offset(const dash_params* p, int32_t b, int32_t kv_head, int32_t row);

/* Stage 0 (Eq. 3, Algorithm 1).  Writes the summaries of chunks [first_block, first_block+num_blocks)
 * of every (batch, KV head) into Kbar, fp32 [batch, h_kv, T_s, head_dim] (T_s = seq_kv / block).
 *   K       keys, dtype p->dtype, strides p->k_stride.
 *   qbar    summary queries, fp32, [h_kv, head_dim] when qbar_chunk_stride == 0, else entry (c, r) at
 *           qbar + c*qbar_chunk_stride + r*head_dim; NULL = zero query = mean pooling.
 *   kv_len  int32 [batch] valid tokens per sequence, or NULL for seq_kv; chunks that are not complete
 *           within kv_len are left untouched.
 * num_blocks < 0 means "to the end".  A summary depends only on its own chunk, so a cache can be
 * extended by calling this for the chunks that completed since the last call. */
int dash_attn_block_summaries(const dash_params* p, const void* K, const float* qbar,
                              int64_t qbar_chunk_stride, const int32_t* kv_len, int32_t first_block,
                              int32_t num_blocks, float* Kbar, void* stream);

/* Stage 1 (Eq. 2, Eq. 4, Algorithm 2, Proposition 1).  For every (batch, KV head, query row):
 * chunk logits against Kbar, the entmax threshold of every query head of the group, the group-averaged
 * weights, the support, and the bias of Proposition 1.
 *   Q        queries; prefill [batch, seq_q, h_q, d] by p->q_stride; decode: token stride unused.
 *   Kbar     fp32 [batch, h_kv, T_s, head_dim].
 *   kv_len   decode only (NULL = seq_kv): the query of sequence b sits at kv_len[b]-1 and its candidates
 *            are the chunks before that position's own chunk.  Must be NULL for prefill.
 *   mask, count, blk_idx, blk_bias   outputs described at the top of the file; blk_idx may be NULL.
 *   tau      optional fp32 [batch, h_q, seq_q] thresholds (in the scaled units of x), NULL to skip;
 *            rows without candidates get 0.
 * A chunk is in the support iff max over the group's heads of (x - tau) > 0. */
int dash_attn_select(const dash_params* p, const void* Q, const float* Kbar, const int32_t* kv_len,
                     uint32_t* mask, int32_t* count, int32_t* blk_idx, float* blk_bias, float* tau,
                     void* workspace, size_t workspace_bytes, void* stream);

/* Stage 2 alone, prefill (Eq. 7 in the form of Proposition 1, Algorithm 3): online-softmax attention of
 * every row over the chunks its mask marks, adding blk_bias to the logits of routed chunks and applying
 * the causal mask inside the row's own chunk.  mask / blk_bias in the layout dash_attn_select writes
 * (any mask obeying it is accepted, e.g. a random one).  O has dtype p->dtype, strides p->o_stride. */
int dash_attn_attend_prefill(const dash_params* p, const void* Q, const void* K, const void* V,
                             const uint32_t* mask, const float* blk_bias, void* O, void* workspace,
                             size_t workspace_bytes, void* stream);

/* Stage 2 alone, decode: one query row per sequence at position kv_len[b]-1, the routed chunk list split
 * across thread blocks along KV and merged (Section 3.5, split-KV variant). */
int dash_attn_attend_decode(const dash_params* p, const void* Q, const void* Kcache, const void* Vcache,
                            const int32_t* kv_len, const int32_t* count, const int32_t* blk_idx,
                            const float* blk_bias, void* O, void* workspace, size_t workspace_bytes,
                            void* stream);

/* dash_attn_attend_decode without any scratch from the caller.  (The paper has no counterpart: this is a
 * packaging variant of the call above, computing exactly the same thing.)
 *
 * Who it is for: callers that cannot hand the library a workspace because they are not allowed to allocate
 * device memory at the point of the call -- a serving loop whose memory plan was frozen at start-up, a plugin
 * inside a host runtime that owns the allocator, code on a path where cudaMalloc's implicit device
 * synchronisation is unacceptable.  They still pass the inputs and the output; the split-KV partial results
 * (m, l, O per split and head), which dash_attn_attend_decode keeps in the workspace, go to a fixed 4 MiB
 * device array that is part of the library image (every GPU that loads the library holds it until exit).
 *
 * Limits and rules:
 *   - It always runs the CUDA-core split kernel and a separate merge kernel (the kernels that serve fp32 and
 *     the shapes the tensor-core decode kernel does not take), for every dtype: the result is the one
 *     dash_attn_attend_decode gives, but for bf16 shapes that call is faster (TMA / tcgen05, merge fused in).
 *   - The partials need batch * h_q * n_split * (head_dim + 2) floats, where the split count n_split is chosen
 *     by the library from the problem size and the SM count and is never more than 32 (more than 16 only
 *     for caches beyond 2^19 tokens).  A problem with
 *     batch * h_q * 32 * (head_dim + 2) * 4 bytes <= 4 MiB therefore always fits; a larger one may or may not,
 *     and when it does not the call returns DASH_ERR_TOO_LARGE and nothing is enqueued.
 *   - The call allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).  The first call
 *     on each device looks up the array's device address (a host-side query, no allocation); make that first
 *     call before any stream capture begins.
 *   - All calls on a device share the one array.  Every slot a call reads it has written itself first, so
 *     earlier contents never matter, but two calls that overlap on the GPU (different streams) race: keep
 *     calls to this entry point ordered on one stream or otherwise serialised.
 *   - No status word: argument errors are returned synchronously as for the other entry points. */
int dash_attn_attend_decode_static(const dash_params* p, const void* Q, const void* Kcache, const void* Vcache,
                                   const int32_t* kv_len, const int32_t* count, const int32_t* blk_idx,
                                   const float* blk_bias, void* O, void* stream);

/* Backward of Stage 2 alone, prefill, with the routing held fixed (Section 3.5: the backward pass reuses the forward
 * pass's bit mask, which the sparse alpha-entmax Jacobian permits -- appendix "The alpha-entmax mapping"; Eq. 7 in the
 * form of Proposition 1 is what is differentiated).  For L = sum(O * dO) and logits l_j = <q,k_j>/sqrt(d) + bias_c(j):
 *   dQ     gradient w.r.t. Q, dtype p->dtype, strides p->q_stride (every row is written).
 *   dK,dV  gradients w.r.t. K and V, fp32, contiguous [batch, seq_kv, h_kv, head_dim]; zeroed, then accumulated
 *          (tokens no row attends stay zero).
 *   dbias  gradient w.r.t. every entry of blk_bias, fp32, in the layout of blk_bias (entries outside a row's count
 *          stay zero): the quantity a backward of Stage 1 continues from.
 *   dO     incoming gradient of O, dtype p->dtype, strides p->o_stride.
 * mask / blk_bias as written by dash_attn_select for the same parameters.  This is a correctness path on CUDA cores
 * (one warp per row and head, fp32 atomics for dK / dV / dbias, so their last bits vary from run to run); it needs
 * no workspace.  dash_attn_bwd_select_prefill and dash_attn_bwd_block_summaries carry dbias on through the routing. */
int dash_attn_bwd_attend_prefill(const dash_params* p, const void* Q, const void* K, const void* V, const void* dO,
                                 const uint32_t* mask, const float* blk_bias, void* dQ, float* dK, float* dV,
                                 float* dbias, void* stream);

/* The same gradients on tensor cores (bf16, head_dim 128, chunks of 64 or 128 tokens, at least two query heads per KV
 * head, causal; anything else returns DASH_ERR_UNSUPPORTED and nothing is enqueued: call dash_attn_bwd_attend_prefill).
 * Five launches: the forward Stage-2 kernel run for its row statistics (log-sum-exp and delta = <O, dO>; O itself is
 * not written, and P enters its P V product as two bf16 terms, so that delta, which the routing's backward amplifies,
 * is accurate to fp32 class), two small kernels over the mask (routed-chunk counts before every mask word; the union
 * of every query tile's mask words), a query-tile-stationary kernel for dQ and dbias, and a key-slice-stationary
 * kernel for dK and dV (no atomics on dQ, dK, dV: every element has one owner and is written whether or not any
 * row attends it; dbias is zeroed and then receives a few atomic adds per entry, whose order cannot change the
 * sum beyond the last bit).  P and dS enter the dQ / dK / dV products rounded to bf16.
 *   bwd_workspace   device scratch of at least dash_attn_bwd_workspace_bytes(p) bytes, 256-byte aligned, owned by the
 *                   caller; it opens with a status word like the forward workspace's (dash_attn_last_status and
 *                   dash_attn_reset_status accept it): a bounded wait that runs out leaves DASH_ERR_TIMEOUT there.
 * Other arguments, layouts and dtypes as for dash_attn_bwd_attend_prefill. */
size_t dash_attn_bwd_workspace_bytes(const dash_params* p);
int dash_attn_bwd_attend_prefill_tc(const dash_params* p, const void* Q, const void* K, const void* V, const void* dO,
                                    const uint32_t* mask, const float* blk_bias, void* dQ, float* dK, float* dV,
                                    float* dbias, void* bwd_workspace, size_t bwd_workspace_bytes, void* stream);

/* Backward of Stage 1 (prefill, causal): carries dbias on through the log-prior bias (Proposition 1), the group average
 * (Section 3.2) and the alpha-entmax of every head (Eq. 2) to the queries and the chunk summaries.  Inside a region
 * of fixed support the entmax Jacobian is diag(s) - s s^T / sum(s) with s = p^(2 - alpha) on the support and zero
 * elsewhere (derived from Eq. 2; the appendix "The alpha-entmax mapping" states that such a closed form exists), so
 * only the routed chunks of a row are visited: the forward pass's list is reused (Section 3.5).
 *   count, blk_idx, tau   as written by dash_attn_select for the same parameters (blk_idx and tau requested).
 *   dbias      fp32, layout of blk_bias: gradient w.r.t. every bias entry (dash_attn_bwd_attend_prefill writes it).
 *   dQ_route   fp32, contiguous [batch, seq_q, h_q, head_dim]: the part of dL/dQ that flows through the routing; the
 *              caller adds it to the Stage-2 part (every row is written, zeros where nothing is routed).
 *   dKbar      fp32 [batch, h_kv, T_s, head_dim]: gradient w.r.t. the summaries; zeroed, then accumulated (atomics).
 * CUDA-core correctness path.  Rows whose support holds a chunk sitting on the threshold have no gradient in the
 * mathematical sense (the map is piecewise differentiable); the kernel then returns the one-sided value of Eq. 2. */
int dash_attn_bwd_select_prefill(const dash_params* p, const void* Q, const float* Kbar, const int32_t* count,
                                 const int32_t* blk_idx, const float* tau, const float* dbias, float* dQ_route,
                                 float* dKbar, void* stream);

/* Backward of Stage 0 (Eq. 3): adds to dK what reaches the keys through their chunk's summary and returns the gradient
 * of the summary query.
 *   qbar / qbar_chunk_stride   as in dash_attn_block_summaries (NULL: mean pooling).
 *   dKbar   fp32 [batch, h_kv, T_s, head_dim].
 *   dK      fp32, contiguous [batch, seq_kv, h_kv, head_dim]: ADDED to (it usually already holds the Stage-2 part).
 *   dqbar   fp32, shape of qbar (zeroed, then accumulated); ignored when qbar is NULL. */
int dash_attn_bwd_block_summaries(const dash_params* p, const void* K, const float* qbar, int64_t qbar_chunk_stride,
                                  const float* dKbar, float* dK, float* dqbar, void* stream);

/* Whole prefill forward: Stage 0 (skipped when Kbar is given), Stage 1, Stage 2.
 *   qbar / qbar_chunk_stride as in dash_attn_block_summaries (used only when Kbar == NULL).
 *   Kbar      NULL: summaries are computed into the workspace; else used as given.
 *   mask_out  optional uint32 [batch, h_kv, seq_q, W]; NULL keeps the mask in the workspace. */
int dash_attn_fwd_prefill(const dash_params* p, const void* Q, const void* K, const void* V,
                          const float* qbar, int64_t qbar_chunk_stride, const float* Kbar, void* O,
                          uint32_t* mask_out, void* workspace, size_t workspace_bytes, void* stream);

/* Whole decode step: Stage 1 for the one new row of every sequence against the summary cache, then the
 * split-KV Stage 2 over the selected chunks of the KV cache.  Kbar must hold the summaries of every chunk
 * that is complete within kv_len[b]-1 tokens (dash_attn_block_summaries keeps it up to date). */
int dash_attn_fwd_decode(const dash_params* p, const void* Q, const void* Kcache, const void* Vcache,
                         const float* Kbar, const int32_t* kv_len, void* O, void* workspace,
                         size_t workspace_bytes, void* stream);

/* Paged KV cache (the paper leaves the serving integration open; this is the decode path over a block-table cache as
 * serving engines keep it, computing exactly what the contiguous calls compute).
 *   Kpool, Vpool  pools of pages, [num_pages, page_size, h_kv, head_dim]: p->k_stride / p->v_stride are the element
 *                 strides of (page, token inside the page, head).
 *   page_table    int32 [batch, max_pages] (device): physical page of every logical page of every sequence; entries
 *                 behind a sequence's kv_len are never read.
 *   page_size     tokens per page: a multiple of 64 and of p->block, so that neither a chunk nor a 64-token tile
 *                 straddles a page;  p->seq_kv must equal max_pages * page_size (the logical capacity).
 * The summary cache Kbar stays contiguous per sequence ([batch, h_kv, T_s, head_dim], indexed by logical chunk), so
 * Stage 1 is untouched; dash_attn_block_summaries_paged fills it from the paged keys, dash_attn_fwd_decode_paged is
 * dash_attn_fwd_decode with the K / V tiles fetched page by page (one TMA box per 64-token tile, its outermost
 * coordinate the physical page).  Both return DASH_ERR_INVALID_ARG for prefill shapes or a page size that breaks
 * the rules above. */
int dash_attn_block_summaries_paged(const dash_params* p, const void* Kpool, const int32_t* page_table,
                                    int32_t page_size, int32_t max_pages, int32_t num_pages, const float* qbar,
                                    int64_t qbar_chunk_stride, const int32_t* kv_len, int32_t first_block,
                                    int32_t num_blocks, float* Kbar, void* stream);
int dash_attn_fwd_decode_paged(const dash_params* p, const void* Q, const void* Kpool, const void* Vpool,
                               const int32_t* page_table, int32_t page_size, int32_t max_pages, int32_t num_pages,
                               const float* Kbar, const int32_t* kv_len, void* O, void* workspace,
                               size_t workspace_bytes, void* stream);

/* Zeroes the status word (enqueued on stream).  Call once after allocating a workspace, and again after an
 * error: the word is sticky (the first error wins), and while it is non-zero the tensor-core kernels launched
 * on that workspace retire without computing, so that one wait that ran out costs one wait limit, not one per
 * thread block; their outputs are then undefined. */
int dash_attn_reset_status(void* workspace, void* stream);

/* Synchronises `stream` and returns the workspace's status word (DASH_OK or a device-side error). */
int dash_attn_last_status(const void* workspace, void* stream);

/* Number of kernel launches this library has enqueued in this process (for launch accounting). */
int64_t dash_attn_launch_count(void);

/* Switches for the test-suite; production code never calls this (process-wide, not thread-safe, defaults restored
 * by (0, 0)).
 *   wait_limit_cycles  SM clock cycles a bounded device-side wait of the prefill attention kernel may spin before it
 *                      gives up with DASH_ERR_TIMEOUT; <= 0 restores the default (2e9, about a second).
 *   skip_own_k_load    1: the tensor-core prefill attention kernel never issues the load of its first K tile, so
 *                      the waits for it run out -- with a short limit this exercises the time-out path (roles leave
 *                      their loops, copies in flight land, tensor memory is freed, the status word is set) without
 *                      hanging or faulting anything. */
void dash_attn_test_hooks(int64_t wait_limit_cycles, int32_t skip_own_k_load);

const char* dash_attn_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* DASH_ATTN_H_ */
