// C ABI of the DashAttention library: argument validation, workspace carving and stage dispatch.
// Every operation is defined in include/dash_attn.h; kernels live in the sibling translation units.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace dash {

// NVTX range around the launches of one stage (a no-op unless a profiler is attached).
struct StageRange {
  explicit StageRange(const char* name) { nvtxRangePushA(name); }
  ~StageRange() { nvtxRangePop(); }
};

static std::atomic<long long> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

TestHooks& test_hooks() {
  static TestHooks hooks;
  return hooks;
}

static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct WorkspaceLayout {
  size_t status, kbar, mask, count, blk_idx, blk_bias, partials, planes, xscratch, total;
};

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

static int check_strides(const long long* s, int dtype) {
  const int mult = dtype == DASH_BF16 ? 8 : 4;
  for (int k = 0; k < 3; ++k)
    if (s[k] < 0 || s[k] % mult != 0) return 0;
  return 1;
}

// Validates p and fills the derived description.  Returns a dash_status.
static int make_dims(const dash_params* p, Dims* dm) {
  if (!p) return DASH_ERR_INVALID_ARG;
  if (p->struct_size != sizeof(dash_params)) return DASH_ERR_INVALID_ARG;
  if (p->batch <= 0 || p->seq_q <= 0 || p->seq_kv <= 0 || p->h_q <= 0 || p->h_kv <= 0) return DASH_ERR_INVALID_ARG;
  if (p->batch > 65535 || p->h_kv > 65535) return DASH_ERR_INVALID_ARG;
  if (p->h_q % p->h_kv != 0) return DASH_ERR_INVALID_ARG;
  if (p->dtype != DASH_F32 && p->dtype != DASH_BF16) return DASH_ERR_INVALID_ARG;
  if (!(p->alpha > 1.f) || !(p->gamma > 0.f) || !(p->sigma > 0.f)) return DASH_ERR_INVALID_ARG;
  if (!std::isfinite(p->alpha) || !std::isfinite(p->gamma) || !std::isfinite(p->sigma)) return DASH_ERR_INVALID_ARG;
  if (p->local_blocks < 0 || p->local_blocks > (1 << 24)) return DASH_ERR_INVALID_ARG;
  if (p->seq_q != p->seq_kv && p->seq_q != 1) return DASH_ERR_INVALID_ARG;
  const int g_q = p->h_q / p->h_kv;
  if (p->q_to_kv) {
    for (int h = 0; h < p->h_q; ++h)
      if (p->q_to_kv[h] != h / g_q) return DASH_ERR_UNSUPPORTED;
  }
  if (p->head_dim != 64 && p->head_dim != 128) return DASH_ERR_UNSUPPORTED;
  if (p->block != 16 && p->block != 32 && p->block != 64 && p->block != 128) return DASH_ERR_UNSUPPORTED;
  if (g_q != 1 && g_q != 2 && g_q != 4 && g_q != 8 && g_q != 16) return DASH_ERR_UNSUPPORTED;
  if (p->causal != 0 && p->causal != 1) return DASH_ERR_INVALID_ARG;
  if (p->causal == 0 && p->local_blocks != 0) return DASH_ERR_INVALID_ARG;   // the window is a causal notion
  if (p->causal == 0 && p->seq_q == 1 && p->seq_kv != 1) return DASH_ERR_UNSUPPORTED;   // decode is causal by nature
  if (!check_strides((const long long*)p->q_stride, p->dtype) || !check_strides((const long long*)p->k_stride, p->dtype) ||
      !check_strides((const long long*)p->v_stride, p->dtype) || !check_strides((const long long*)p->o_stride, p->dtype))
    return DASH_ERR_INVALID_ARG;

  std::memset(dm, 0, sizeof(*dm));
  dm->batch = p->batch; dm->seq_q = p->seq_q; dm->seq_kv = p->seq_kv;
  dm->h_q = p->h_q; dm->h_kv = p->h_kv; dm->d = p->head_dim; dm->B = p->block; dm->g_q = g_q;
  dm->dtype = p->dtype;
  dm->local_blocks = p->local_blocks;
  dm->causal = p->causal;
  dm->T_s = p->seq_kv / p->block;
  dm->T_a = (p->seq_kv + p->block - 1) / p->block;
  dm->W = (dm->T_a + 31) / 32;
  dm->decode = (p->seq_q == 1 && p->seq_kv != 1) ? 1 : 0;
  dm->e = 1.f / (p->alpha - 1.f);
  dm->e_int = p->alpha == 2.f ? 1 : p->alpha == 1.5f ? 2 : p->alpha == 1.25f ? 4 : 0;
  dm->sm_scale = 1.f / std::sqrt((float)p->head_dim);
  dm->x_scale = (float)((double)p->gamma * ((double)p->alpha - 1.0) / std::sqrt((double)p->head_dim));
  dm->inv_sigma = 1.f / p->sigma;
  for (int k = 0; k < 3; ++k) {
    dm->qs[k] = p->q_stride[k]; dm->ks[k] = p->k_stride[k]; dm->vs[k] = p->v_stride[k]; dm->os[k] = p->o_stride[k];
  }
  if (dm->decode) {
    dm->list_rows = dm->T_s;
  } else if (!dm->causal) {
    dm->list_rows = (long long)p->seq_q * dm->T_s;
  } else {
    const long long n = p->seq_q;
    const long long c = n / p->block;
    dm->list_rows = (long long)p->block * c * (c - 1) / 2 + (n % p->block) * c;
  }
  if (select_smem_bytes(*dm, nullptr) == 0) return DASH_ERR_UNSUPPORTED;  // score rows do not fit on chip
  return DASH_OK;
}

static WorkspaceLayout layout(const Dims& dm) {
  WorkspaceLayout w;
  size_t off = 0;
  w.status = off; off += STATUS_REGION_BYTES;   // status word + arrival counters
  w.kbar = off; off += align256((size_t)dm.batch * dm.h_kv * (size_t)max(dm.T_s, 1) * dm.d * sizeof(float));
  w.mask = off; off += align256((size_t)dm.batch * dm.h_kv * (size_t)dm.seq_q * dm.W * sizeof(uint32_t));
  w.count = off; off += align256((size_t)dm.batch * dm.h_kv * (size_t)dm.seq_q * sizeof(int));
  const size_t cap = (size_t)dm.batch * dm.h_kv * (size_t)(dm.list_rows > 0 ? dm.list_rows : 1);
  w.blk_idx = off; off += align256(cap * sizeof(int));
  w.blk_bias = off; off += align256(cap * sizeof(float));
  w.partials = off; off += align256(dm.decode ? decode_partial_bytes(dm) : 0);
  w.planes = off; off += align256(select_sm100_token_limit(dm) > 0 ? select_sm100_scratch_bytes(dm) : 0);
  w.xscratch = off; off += align256(select_decode_scratch_bytes(dm));
  w.total = off;
  return w;
}

static int check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return DASH_ERR_CUDA;
  static std::atomic<int> cached[64];  // per device: 0 unknown, 1 ok, 2 wrong architecture
  const bool tracked = dev >= 0 && dev < 64;
  if (const int c = tracked ? cached[dev].load(std::memory_order_relaxed) : 0) return c == 1 ? DASH_OK : DASH_ERR_ARCH;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return DASH_ERR_CUDA;
  if (tracked) cached[dev].store(major == 10 ? 1 : 2, std::memory_order_relaxed);
  return major == 10 ? DASH_OK : DASH_ERR_ARCH;
}

static int check_workspace(const Dims& dm, void* ws, size_t bytes, WorkspaceLayout* out) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0) return DASH_ERR_WORKSPACE;
  *out = layout(dm);
  if (bytes < out->total) return DASH_ERR_WORKSPACE;
  return DASH_OK;
}

// Adds the description of a paged KV cache to a decode problem (see the header for the rules).
static int add_paging(Dims* dm, const int32_t* page_table, int page_size, int max_pages, int num_pages) {
  if (!dm->decode) return DASH_ERR_INVALID_ARG;
  if (!page_table || page_size <= 0 || max_pages <= 0 || num_pages <= 0) return DASH_ERR_INVALID_ARG;
  if (page_size % 64 != 0 || page_size % dm->B != 0) return DASH_ERR_INVALID_ARG;
  if ((long long)max_pages * page_size != dm->seq_kv) return DASH_ERR_INVALID_ARG;
  dm->page_table = page_table;
  dm->page_size = page_size;
  dm->max_pages = max_pages;
  dm->num_pages = num_pages;
  return DASH_OK;
}

int validate_params(const dash_params* p, Dims* dm) { return make_dims(p, dm); }
int validate_device() { return check_device(); }

template <typename T> static T* at(void* ws, size_t off) { return reinterpret_cast<T*>(static_cast<char*>(ws) + off); }

static int cuda_status(cudaError_t e) { return e == cudaSuccess ? DASH_OK : DASH_ERR_CUDA; }

static int run_attend_prefill(const Dims& dm, const void* Q, const void* K, const void* V, const uint32_t* mask,
                              const float* blk_bias, void* O, StatusBlock* sb, bool inputs_stable, cudaStream_t st) {
  if (prefill_sm100_supported(dm))
    return cuda_status(launch_attend_prefill_sm100(dm, Q, K, V, mask, blk_bias, O, sb, inputs_stable, st));
  return cuda_status(launch_attend_prefill_generic(dm, Q, K, V, mask, blk_bias, O, st));
}

}  // namespace dash

using namespace dash;

extern "C" {

size_t dash_attn_workspace_bytes(const dash_params* p) {
  Dims dm;
  if (make_dims(p, &dm) != DASH_OK) return 0;
  return layout(dm).total;
}

int64_t dash_attn_list_capacity(const dash_params* p) {
  Dims dm;
  if (make_dims(p, &dm) != DASH_OK) return -1;
  return (int64_t)dm.batch * dm.h_kv * dm.list_rows;
}

int64_t dash_attn_list_offset(const dash_params* p, int32_t b, int32_t kv_head, int32_t row) {
  Dims dm;
  if (make_dims(p, &dm) != DASH_OK) return -1;
  if (b < 0 || b >= dm.batch || kv_head < 0 || kv_head >= dm.h_kv || row < 0 || row >= dm.seq_q) return -1;
  return ((int64_t)b * dm.h_kv + kv_head) * dm.list_rows + list_row_offset(dm, row);
}

int dash_attn_block_summaries(const dash_params* p, const void* K, const float* qbar, int64_t qbar_chunk_stride,
                              const int32_t* kv_len, int32_t first_block, int32_t num_blocks, float* Kbar,
                              void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (!K || !aligned16(K)) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && (!Kbar || !aligned16(Kbar))) return DASH_ERR_INVALID_ARG;  // no complete chunk: nothing to write
  if (qbar && (!aligned16(qbar) || qbar_chunk_stride < 0 || qbar_chunk_stride % 4 != 0)) return DASH_ERR_INVALID_ARG;
  if (first_block < 0 || first_block > dm.T_s) return DASH_ERR_INVALID_ARG;
  if (num_blocks < 0) num_blocks = dm.T_s - first_block;
  if (first_block + num_blocks > dm.T_s) return DASH_ERR_INVALID_ARG;
  if ((rc = check_device()) != DASH_OK) return rc;
  StageRange nv("dash_attn: stage 0 summaries");
  return cuda_status(launch_summaries(dm, K, qbar, qbar_chunk_stride, kv_len, first_block, num_blocks, Kbar, nullptr,
                                      (cudaStream_t)stream));
}

int dash_attn_block_summaries_paged(const dash_params* p, const void* Kpool, const int32_t* page_table,
                                    int32_t page_size, int32_t max_pages, int32_t num_pages, const float* qbar,
                                    int64_t qbar_chunk_stride, const int32_t* kv_len, int32_t first_block,
                                    int32_t num_blocks, float* Kbar, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if ((rc = add_paging(&dm, page_table, page_size, max_pages, num_pages)) != DASH_OK) return rc;
  if (!Kpool || !aligned16(Kpool)) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && (!Kbar || !aligned16(Kbar))) return DASH_ERR_INVALID_ARG;
  if (qbar && (!aligned16(qbar) || qbar_chunk_stride < 0 || qbar_chunk_stride % 4 != 0)) return DASH_ERR_INVALID_ARG;
  if (first_block < 0 || first_block > dm.T_s) return DASH_ERR_INVALID_ARG;
  if (num_blocks < 0) num_blocks = dm.T_s - first_block;
  if (first_block + num_blocks > dm.T_s) return DASH_ERR_INVALID_ARG;
  if ((rc = check_device()) != DASH_OK) return rc;
  StageRange nv("dash_attn: stage 0 summaries");
  return cuda_status(launch_summaries(dm, Kpool, qbar, qbar_chunk_stride, kv_len, first_block, num_blocks, Kbar, nullptr,
                                      (cudaStream_t)stream));
}

int dash_attn_select(const dash_params* p, const void* Q, const float* Kbar, const int32_t* kv_len, uint32_t* mask,
                     int32_t* count, int32_t* blk_idx, float* blk_bias, float* tau, void* workspace,
                     size_t workspace_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (!Q || !mask || !count || !aligned16(Q)) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && (!Kbar || !aligned16(Kbar) || !blk_bias)) return DASH_ERR_INVALID_ARG;
  if (!dm.decode && kv_len) return DASH_ERR_INVALID_ARG;
  WorkspaceLayout wl;
  if ((rc = check_workspace(dm, workspace, workspace_bytes, &wl)) != DASH_OK) return rc;
  if ((rc = check_device()) != DASH_OK) return rc;
  StageRange nv("dash_attn: stage 1 routing");
  return cuda_status(launch_select(dm, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau,
                                   at<void>(workspace, wl.planes), at<float>(workspace, wl.xscratch), at<StatusBlock>(workspace, wl.status),
                                   (cudaStream_t)stream));
}

int dash_attn_attend_prefill(const dash_params* p, const void* Q, const void* K, const void* V, const uint32_t* mask,
                             const float* blk_bias, void* O, void* workspace, size_t workspace_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (dm.decode) return DASH_ERR_INVALID_ARG;
  if (!Q || !K || !V || !mask || !O) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && !blk_bias) return DASH_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return DASH_ERR_INVALID_ARG;
  WorkspaceLayout wl;
  if ((rc = check_workspace(dm, workspace, workspace_bytes, &wl)) != DASH_OK) return rc;
  if ((rc = check_device()) != DASH_OK) return rc;
  StageRange nv("dash_attn: stage 2 prefill attention");
  // the kernel before this one on the stream is unknown here and may have produced Q, K or V
  return run_attend_prefill(dm, Q, K, V, mask, blk_bias, O, at<StatusBlock>(workspace, wl.status), false,
                            (cudaStream_t)stream);
}

int dash_attn_attend_decode(const dash_params* p, const void* Q, const void* Kcache, const void* Vcache,
                            const int32_t* kv_len, const int32_t* count, const int32_t* blk_idx,
                            const float* blk_bias, void* O, void* workspace, size_t workspace_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (!dm.decode) return DASH_ERR_INVALID_ARG;
  if (!Q || !Kcache || !Vcache || !count || !O) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && (!blk_idx || !blk_bias)) return DASH_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(Kcache) || !aligned16(Vcache) || !aligned16(O)) return DASH_ERR_INVALID_ARG;
  WorkspaceLayout wl;
  if ((rc = check_workspace(dm, workspace, workspace_bytes, &wl)) != DASH_OK) return rc;
  if ((rc = check_device()) != DASH_OK) return rc;
  StageRange nv("dash_attn: stage 2 decode attention");
  return cuda_status(launch_attend_decode_ex(dm, Q, Kcache, Vcache, kv_len, count, blk_idx, blk_bias, O,
                                             at<float>(workspace, wl.partials), at<StatusBlock>(workspace, wl.status),
                                             (cudaStream_t)stream));
}

int dash_attn_bwd_attend_prefill(const dash_params* p, const void* Q, const void* K, const void* V, const void* dO,
                                 const uint32_t* mask, const float* blk_bias, void* dQ, float* dK, float* dV,
                                 float* dbias, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (dm.decode) return DASH_ERR_INVALID_ARG;
  if (!Q || !K || !V || !dO || !mask || !dQ || !dK || !dV) return DASH_ERR_INVALID_ARG;
  if (dm.list_rows > 0 && (!blk_bias || !dbias)) return DASH_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dO) || !aligned16(dQ) || !aligned16(dK) ||
      !aligned16(dV))
    return DASH_ERR_INVALID_ARG;
  if ((rc = check_device()) != DASH_OK) return rc;
  StageRange nv("dash_attn: stage 2 prefill attention, backward");
  return cuda_status(launch_attend_prefill_bwd_generic(dm, Q, K, V, dO, mask, blk_bias, dQ, dK, dV, dbias,
                                                       (cudaStream_t)stream));
}

// Layout of the backward scratch: status region, then lse2 and delta [batch][KV head][query tile][128 rows], then the
// routed-chunk prefix counts [batch * h_kv * seq_q][W].
struct BwdLayout {
  size_t status, lse2, delta, prefix, total;
};
static BwdLayout bwd_layout(const Dims& dm) {
  auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
  BwdLayout l;
  l.status = 0;
  size_t at = up(STATUS_REGION_BYTES);
  const int tq = std::max(1, std::min(128 / std::max(dm.g_q, 1), dm.B));
  const size_t rows = (size_t)dm.batch * dm.h_kv * (size_t)((dm.seq_q + tq - 1) / tq) * 128;
  l.lse2 = at; at = up(at + rows * sizeof(float));
  l.delta = at; at = up(at + rows * sizeof(float));
  // prefix counts [batch * h_kv * seq_q][W], then the tiles' mask unions [batch * h_kv][query tile][W]
  l.prefix = at; at = up(at + ((size_t)dm.batch * dm.h_kv * dm.seq_q + (size_t)dm.batch * dm.h_kv * ((dm.seq_q + tq - 1) / tq)) *
                                  (size_t)dm.W * sizeof(int));
  l.total = at;
  return l;
}

size_t dash_attn_bwd_workspace_bytes(const dash_params* p) {
  Dims dm;
  if (make_dims(p, &dm) != DASH_OK || dm.decode) return 0;
  return bwd_layout(dm).total;
}

int dash_attn_bwd_attend_prefill_tc(const dash_params* p, const void* Q, const void* K, const void* V, const void* dO,
                                    const uint32_t* mask, const float* blk_bias, void* dQ, float* dK, float* dV,
                                    float* dbias, void* bwd_workspace, size_t bwd_workspace_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (dm.decode) return DASH_ERR_INVALID_ARG;
  if (!Q || !K || !V || !dO || !mask || !dQ || !dK || !dV) return DASH_ERR_INVALID_ARG;
  if (dm.list_rows > 0 && (!blk_bias || !dbias)) return DASH_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dO) || !aligned16(dQ) || !aligned16(dK) ||
      !aligned16(dV))
    return DASH_ERR_INVALID_ARG;
  const BwdLayout l = bwd_layout(dm);
  if (!bwd_workspace || (reinterpret_cast<uintptr_t>(bwd_workspace) & 255) != 0) return DASH_ERR_WORKSPACE;
  if (bwd_workspace_bytes < l.total) return DASH_ERR_WORKSPACE;
  if ((rc = check_device()) != DASH_OK) return rc;
  if (!prefill_bwd_sm100_supported(dm)) return DASH_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  StageRange nv("dash_attn: stage 2 prefill attention, backward (tensor cores)");
  const size_t list_bytes = (size_t)dm.batch * dm.h_kv * (size_t)dm.list_rows * sizeof(float);
  if (list_bytes > 0) {
    if ((rc = cuda_status(cudaMemsetAsync(dbias, 0, list_bytes, st))) != DASH_OK) return rc;
  }
  return cuda_status(launch_attend_prefill_bwd_sm100(dm, Q, K, V, dO, mask, blk_bias, at<float>(bwd_workspace, l.lse2),
                                                     at<float>(bwd_workspace, l.delta), at<int>(bwd_workspace, l.prefix),
                                                     dQ, dK, dV, dbias, at<StatusBlock>(bwd_workspace, l.status), st));
}

int dash_attn_bwd_select_prefill(const dash_params* p, const void* Q, const float* Kbar, const int32_t* count,
                                 const int32_t* blk_idx, const float* tau, const float* dbias, float* dQ_route,
                                 float* dKbar, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (dm.decode || !dm.causal) return DASH_ERR_UNSUPPORTED;
  if (!Q || !count || !dQ_route || !aligned16(Q)) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && (!Kbar || !blk_idx || !tau || !dbias || !dKbar)) return DASH_ERR_INVALID_ARG;
  if ((rc = check_device()) != DASH_OK) return rc;
  StageRange nv("dash_attn: stage 1 routing, backward");
  return cuda_status(launch_route_bwd(dm, Q, Kbar, count, blk_idx, tau, dbias, dQ_route, dKbar, (cudaStream_t)stream));
}

int dash_attn_bwd_block_summaries(const dash_params* p, const void* K, const float* qbar, int64_t qbar_chunk_stride,
                                  const float* dKbar, float* dK, float* dqbar, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (dm.decode) return DASH_ERR_UNSUPPORTED;
  if (!K || !dK || !aligned16(K)) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && !dKbar) return DASH_ERR_INVALID_ARG;
  if (qbar && (qbar_chunk_stride < 0 || qbar_chunk_stride % 4 != 0)) return DASH_ERR_INVALID_ARG;
  if ((rc = check_device()) != DASH_OK) return rc;
  const size_t dq_bytes = !qbar ? 0 : (qbar_chunk_stride == 0 ? (size_t)dm.h_kv * dm.d
                                                               : (size_t)dm.T_s * (size_t)qbar_chunk_stride) * sizeof(float);
  StageRange nv("dash_attn: stage 0 summaries, backward");
  return cuda_status(launch_summaries_bwd(dm, K, qbar, qbar_chunk_stride, dKbar, dK, qbar ? dqbar : nullptr, dq_bytes,
                                          (cudaStream_t)stream));
}

int dash_attn_fwd_prefill(const dash_params* p, const void* Q, const void* K, const void* V, const float* qbar,
                          int64_t qbar_chunk_stride, const float* Kbar, void* O, uint32_t* mask_out, void* workspace,
                          size_t workspace_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (dm.decode) return DASH_ERR_INVALID_ARG;
  if (!Q || !K || !V || !O) return DASH_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return DASH_ERR_INVALID_ARG;
  if (Kbar && !aligned16(Kbar)) return DASH_ERR_INVALID_ARG;
  if (qbar && (!aligned16(qbar) || qbar_chunk_stride < 0 || qbar_chunk_stride % 4 != 0)) return DASH_ERR_INVALID_ARG;
  WorkspaceLayout wl;
  if ((rc = check_workspace(dm, workspace, workspace_bytes, &wl)) != DASH_OK) return rc;
  if ((rc = check_device()) != DASH_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  StatusBlock* sb = at<StatusBlock>(workspace, wl.status);
  const float* kb = Kbar;
  bool planes_ready = false;
  if (!kb) {
    float* kbw = at<float>(workspace, wl.kbar);
    // the tensor-core routing kernel reads Kbar as three bf16 planes: the summary kernel writes them directly
    void* planes = select_sm100_token_limit(dm) > 0 ? at<void>(workspace, wl.planes) : nullptr;
    StageRange nv("dash_attn: stage 0 summaries");
    if ((rc = cuda_status(launch_summaries(dm, K, qbar, qbar_chunk_stride, nullptr, 0, dm.T_s, kbw, planes, st))) != DASH_OK)
      return rc;
    kb = kbw;
    planes_ready = planes != nullptr && dm.T_s > 0;
  }
  uint32_t* mask = mask_out ? mask_out : at<uint32_t>(workspace, wl.mask);
  float* bias = at<float>(workspace, wl.blk_bias);
  {
    StageRange nv("dash_attn: stage 1 routing");
    if ((rc = cuda_status(launch_select(dm, Q, kb, nullptr, mask, at<int>(workspace, wl.count), nullptr, bias, nullptr,
                                        at<void>(workspace, wl.planes), at<float>(workspace, wl.xscratch), sb, st,
                                        planes_ready))) != DASH_OK)
      return rc;
  }
  StageRange nv("dash_attn: stage 2 prefill attention");
  // the kernel before Stage 2 is this call's own routing kernel, which writes none of Q, K, V
  return run_attend_prefill(dm, Q, K, V, mask, bias, O, sb, true, st);
}

int dash_attn_fwd_decode(const dash_params* p, const void* Q, const void* Kcache, const void* Vcache,
                         const float* Kbar, const int32_t* kv_len, void* O, void* workspace, size_t workspace_bytes,
                         void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if (!dm.decode) return DASH_ERR_INVALID_ARG;
  if (!Q || !Kcache || !Vcache || !O) return DASH_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(Kcache) || !aligned16(Vcache) || !aligned16(O)) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && (!Kbar || !aligned16(Kbar))) return DASH_ERR_INVALID_ARG;
  WorkspaceLayout wl;
  if ((rc = check_workspace(dm, workspace, workspace_bytes, &wl)) != DASH_OK) return rc;
  if ((rc = check_device()) != DASH_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  StatusBlock* sb = at<StatusBlock>(workspace, wl.status);
  int* count = at<int>(workspace, wl.count);
  int* idx = at<int>(workspace, wl.blk_idx);
  float* bias = at<float>(workspace, wl.blk_bias);
  {
    StageRange nv("dash_attn: stage 1 routing");
    if ((rc = cuda_status(launch_select(dm, Q, Kbar, kv_len, at<uint32_t>(workspace, wl.mask), count, idx, bias, nullptr,
                                        at<void>(workspace, wl.planes), at<float>(workspace, wl.xscratch), sb, st))) != DASH_OK)
      return rc;
  }
  StageRange nv("dash_attn: stage 2 decode attention");
  return cuda_status(launch_attend_decode_ex(dm, Q, Kcache, Vcache, kv_len, count, idx, bias, O,
                                             at<float>(workspace, wl.partials), sb, st));
}

int dash_attn_fwd_decode_paged(const dash_params* p, const void* Q, const void* Kpool, const void* Vpool,
                               const int32_t* page_table, int32_t page_size, int32_t max_pages, int32_t num_pages,
                               const float* Kbar, const int32_t* kv_len, void* O, void* workspace,
                               size_t workspace_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(p, &dm);
  if (rc != DASH_OK) return rc;
  if ((rc = add_paging(&dm, page_table, page_size, max_pages, num_pages)) != DASH_OK) return rc;
  if (!Q || !Kpool || !Vpool || !O) return DASH_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(Kpool) || !aligned16(Vpool) || !aligned16(O)) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && (!Kbar || !aligned16(Kbar))) return DASH_ERR_INVALID_ARG;
  WorkspaceLayout wl;
  if ((rc = check_workspace(dm, workspace, workspace_bytes, &wl)) != DASH_OK) return rc;
  if ((rc = check_device()) != DASH_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  StatusBlock* sb = at<StatusBlock>(workspace, wl.status);
  int* count = at<int>(workspace, wl.count);
  int* idx = at<int>(workspace, wl.blk_idx);
  float* bias = at<float>(workspace, wl.blk_bias);
  {
    // Stage 1 reads the summary cache only, which is indexed by logical chunk: paging does not reach it
    StageRange nv("dash_attn: stage 1 routing");
    if ((rc = cuda_status(launch_select(dm, Q, Kbar, kv_len, at<uint32_t>(workspace, wl.mask), count, idx, bias, nullptr,
                                        at<void>(workspace, wl.planes), at<float>(workspace, wl.xscratch), sb, st))) != DASH_OK)
      return rc;
  }
  StageRange nv("dash_attn: stage 2 decode attention");
  return cuda_status(launch_attend_decode_ex(dm, Q, Kpool, Vpool, kv_len, count, idx, bias, O,
                                             at<float>(workspace, wl.partials), sb, st));
}

int dash_attn_reset_status(void* workspace, void* stream) {
  if (!workspace) return DASH_ERR_WORKSPACE;
  return cuda_status(cudaMemsetAsync(workspace, 0, STATUS_REGION_BYTES, (cudaStream_t)stream));
}

int dash_attn_last_status(const void* workspace, void* stream) {
  if (!workspace) return DASH_ERR_WORKSPACE;
  int st = 0;
  if (cudaMemcpyAsync(&st, workspace, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
    return DASH_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return DASH_ERR_CUDA;
  return st;
}

int64_t dash_attn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

void dash_attn_test_hooks(int64_t wait_limit_cycles, int32_t skip_own_k_load) {
  TestHooks& h = test_hooks();
  h.wait_limit_cycles = wait_limit_cycles > 0 ? wait_limit_cycles : TestHooks().wait_limit_cycles;
  h.skip_own_k_load = skip_own_k_load ? 1 : 0;
}

const char* dash_attn_strerror(int status) {
  switch (status) {
    case DASH_OK: return "ok";
    case DASH_ERR_INVALID_ARG: return "invalid argument";
    case DASH_ERR_UNSUPPORTED: return "unsupported configuration";
    case DASH_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case DASH_ERR_CAPACITY: return "device-side capacity overrun";
    case DASH_ERR_CUDA: return "CUDA call failed";
    case DASH_ERR_ARCH: return "device is not compute capability 10.x";
    case DASH_ERR_TIMEOUT: return "device-side bounded wait ran out";
    case DASH_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of a *_static entry point";
    default: return "unknown status";
  }
}

}  // extern "C"
