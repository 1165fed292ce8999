// Stage 2, decode: split-KV attention of one query row per sequence over its routed chunks
// (Eq. 7 / Proposition 1; Algorithm 3; the split-KV variant of Section 3.5).
//
// The routed-chunk list of every (batch, KV head) plus the row's own (partial) chunk is cut into
// n_split contiguous ranges, one thread block each; inside a block the four warps take chunks
// round-robin.  A warp keeps the online-softmax state (m, l, O) of all g_q heads of the group; lanes own
// keys for the logits and head_dim slices for the output.  Every warp's state is merged in shared
// memory, every block writes one partial (m, l, O) per head, and a second kernel merges the partials in
// split order, so results do not depend on scheduling.  Only the selected chunks' K and V rows are read.
#include <mutex>

#include "common.cuh"

namespace dash {

constexpr int DEC_WARPS = 4;
constexpr int DEC_MAX_SPLITS = 32;

static bool decode_use_sm100(const Dims& dm) {
  const int need = decode_sm100_min_splits(dm);
  return need > 0 && need <= DEC_MAX_SPLITS;
}

// Split count: thread blocks are handed out in waves of one per SM (the tensor-core kernel fills an SM's
// shared memory), so the time is about ceil(groups * s / SMs) waves of (1/s of a group's work + a fixed cost per
// block, about 2 % of a long group's work: list staging, first loads, partial write).  At 128 groups on 148 SMs
// s = 5 leaves a fifth wave a third full, s = 8 fills seven waves almost exactly (measured: 0.155 vs 0.150 ms).
// SM count of the current device, cached per device (a process may drive several GPUs).
static int current_sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  const bool tracked = dev >= 0 && dev < 64;
  int n = tracked ? cached[dev].load(std::memory_order_relaxed) : 0;
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  if (tracked) cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

int decode_num_splits(const Dims& dm) {
  const int n_sm = current_sm_count();
  const int groups = dm.batch * dm.h_kv;
  int lo = 1;
  if (decode_use_sm100(dm)) lo = max(lo, decode_sm100_min_splits(dm));   // a block owns at most 512 sub-blocks there
  const int hi = max(lo, min(DEC_MAX_SPLITS, 16));
  int best = lo;
  double best_cost = 1e30;
  for (int s = lo; s <= hi; ++s) {
    const long long waves = ((long long)groups * s + n_sm - 1) / n_sm;
    const double cost = (double)waves * (1.0 / s + 0.02);
    if (cost < best_cost - 1e-12) { best_cost = cost; best = s; }
  }
  return best;
}

size_t decode_partial_bytes(const Dims& dm) {
  return (size_t)dm.batch * dm.h_q * decode_num_splits(dm) * (dm.d + 2) * sizeof(float);
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(DEC_WARPS * 32)
decode_split_kernel(Dims dm, int n_split, const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                    const int* __restrict__ kv_len, const int* __restrict__ count,
                    const int* __restrict__ blk_idx, const float* __restrict__ blk_bias,
                    float* __restrict__ partials, StatusBlock* sb) {
  constexpr int VPL = D / 32;
  // the merge buffer reuses the query / probability staging space once the main loop is over
  constexpr int QS_N = G * D, PS_N = DEC_WARPS * 32 * G, RED_N = DEC_WARPS * G * (D + 2);
  __shared__ __align__(16) float sm[(QS_N + PS_N > RED_N) ? (QS_N + PS_N) : RED_N];
  float (*qs)[D] = reinterpret_cast<float (*)[D]>(sm);
  float (*ps)[32][G] = reinterpret_cast<float (*)[32][G]>(sm + QS_N);
  float (*red)[G][D + 2] = reinterpret_cast<float (*)[G][D + 2]>(sm);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, r = blockIdx.y, b = blockIdx.z;

  chain_wait();
  chain_release();
  int L = kv_len ? kv_len[b] : dm.seq_kv;
  L = max(1, min(L, dm.seq_kv));
  const int c_own = (L - 1) / dm.B;
  const long long grp = (long long)b * dm.h_kv + r;
  int n_routed = count[grp];
  DASH_CHECK(n_routed >= 0 && n_routed <= min(c_own, dm.T_s), sb, 400, n_routed = 0);
  const int n_items = n_routed + 1;
  const int per = (n_items + n_split - 1) / n_split;
  const int lo = split * per, hi = min(n_items, lo + per);

  for (int idx = tid; idx < G * D; idx += DEC_WARPS * 32) {
    const int g = idx / D, k = idx % D;
    qs[g][k] = to_f32<T>(Q[(long long)b * dm.qs[0] + (long long)(r * G + g) * dm.qs[2] + k]) * dm.sm_scale;
  }
  __syncthreads();

  const long long loff = grp * dm.list_rows;

  float m[G], l[G], acc[G][VPL];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[g][v] = 0.f;
  }

  for (int it = lo + warp; it < hi; it += DEC_WARPS) {
    int c, t_end;
    float bias;
    if (it < n_routed) {
      c = blk_idx[loff + it];
      bias = blk_bias[loff + it];
      DASH_CHECK(c >= 0 && c < c_own, sb, 401, continue);       // routed and window chunks precede the own chunk
      t_end = (c + 1) * dm.B;
    } else {
      c = c_own; bias = 0.f; t_end = L;
    }
    // the chunk's rows: token t of the chunk sits at kbase + t * stride (contiguous cache or inside one page)
    int cfirst, ctok;
    kv_locate(dm, b, c * dm.B, &cfirst, &ctok);
    DASH_CHECK(!dm.page_table || (unsigned)cfirst < (unsigned)dm.num_pages, sb, 402, continue);   // a page id outside the pool
    const T* kbase = K + (long long)cfirst * dm.ks[0] + (long long)r * dm.ks[2] + (long long)(ctok - c * dm.B) * dm.ks[1];
    const T* vbase = V + (long long)cfirst * dm.vs[0] + (long long)r * dm.vs[2] + (long long)(ctok - c * dm.B) * dm.vs[1];
    for (int t0 = c * dm.B; t0 < t_end; t0 += 32) {
      const int t = t0 + lane;
      float s[G];
#pragma unroll
      for (int g = 0; g < G; ++g) s[g] = 0.f;
      if (t < t_end) {
        const T* kp = kbase + (long long)t * dm.ks[1];
#pragma unroll 4
        for (int k = 0; k < D; k += 4) {
          const float4 kv = load4(kp + k);
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float4 qv = *reinterpret_cast<const float4*>(&qs[g][k]);
            s[g] = fmaf(qv.x, kv.x, s[g]); s[g] = fmaf(qv.y, kv.y, s[g]);
            s[g] = fmaf(qv.z, kv.z, s[g]); s[g] = fmaf(qv.w, kv.w, s[g]);
          }
        }
      }
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float sg = (t < t_end) ? s[g] + bias : -INFINITY;
        const float mt = fmaxf(m[g], warp_max(sg));
        const float corr = __expf(m[g] - mt);
        const float p = (t < t_end) ? __expf(sg - mt) : 0.f;
        l[g] = l[g] * corr + p;  // per-lane partial sum; reduced across lanes at the end
#pragma unroll
        for (int v = 0; v < VPL; ++v) acc[g][v] *= corr;
        ps[warp][lane][g] = p;
        m[g] = mt;
      }
      __syncwarp();
      const int nt = min(32, t_end - t0);
      for (int u = 0; u < nt; ++u) {
        const T* vp = vbase + (long long)(t0 + u) * dm.vs[1] + lane * VPL;
        float vv[VPL];
        if constexpr (VPL == 4) {
          const float4 f = load4(vp);
          vv[0] = f.x; vv[1] = f.y; vv[2] = f.z; vv[3] = f.w;
        } else {
          vv[0] = to_f32<T>(vp[0]); vv[1] = to_f32<T>(vp[1]);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const float pu = ps[warp][u][g];
#pragma unroll
          for (int v = 0; v < VPL; ++v) acc[g][v] = fmaf(pu, vv[v], acc[g][v]);
        }
      }
      __syncwarp();
    }
  }

  // merge the four warps, then write one partial per head
  __syncthreads();
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const float lsum = warp_sum(l[g]);
    if (lane == 0) { red[warp][g][0] = m[g]; red[warp][g][1] = lsum; }
#pragma unroll
    for (int v = 0; v < VPL; ++v) red[warp][g][2 + lane * VPL + v] = acc[g][v];
  }
  __syncthreads();
  for (int idx = tid; idx < G * (D + 2); idx += DEC_WARPS * 32) {
    const int g = idx / (D + 2), k = idx % (D + 2);
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, red[w][g][0]);
    float out;
    if (k == 0) {
      out = M;
    } else {
      out = 0.f;
      if (M > -INFINITY) {
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) out += red[w][g][k] * __expf(red[w][g][0] - M);
      }
    }
    partials[(((long long)b * dm.h_q + r * G + g) * n_split + split) * (D + 2) + k] = out;
  }
}

// One warp per (batch, query head): merge the split partials in split order and normalise.
template <typename T, int D>
__global__ void decode_merge_kernel(Dims dm, int n_split, const float* __restrict__ partials, T* __restrict__ O) {
  constexpr int VPL = D / 32;
  const int lane = threadIdx.x & 31;
  const long long bh = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (bh >= (long long)dm.batch * dm.h_q) return;
  chain_wait();
  chain_release();
  const float* p = partials + bh * n_split * (D + 2);
  float M = -INFINITY;
  for (int s = 0; s < n_split; ++s) M = fmaxf(M, p[s * (D + 2)]);
  float Lsum = 0.f, acc[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) acc[v] = 0.f;
  for (int s = 0; s < n_split; ++s) {
    const float ms = p[s * (D + 2)];
    if (ms == -INFINITY) continue;
    const float w = __expf(ms - M);
    Lsum += w * p[s * (D + 2) + 1];
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[v] += w * p[s * (D + 2) + 2 + lane * VPL + v];
  }
  const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
  const int b = (int)(bh / dm.h_q), h = (int)(bh % dm.h_q);
  T* op = O + (long long)b * dm.os[0] + (long long)h * dm.os[2] + lane * VPL;
#pragma unroll
  for (int v = 0; v < VPL; ++v) op[v] = from_f32<T>(acc[v] * inv);
}

template <typename T, int D>
static cudaError_t launch_dec(const Dims& dm, const void* Q, const void* K, const void* V, const int* kv_len,
                              const int* count, const int* blk_idx, const float* blk_bias, void* O,
                              float* partials, StatusBlock* sb, cudaStream_t st) {
  const int ns = decode_num_splits(dm);
  dim3 grid(ns, dm.h_kv, dm.batch);
  cudaError_t e = cudaSuccess;
#define DASH_DEC(G)                                                                                              \
  e = launch_chained(decode_split_kernel<T, D, G>, grid, dim3(DEC_WARPS * 32), 0, st, dm, ns, (const T*)Q,       \
                     (const T*)K, (const T*)V, kv_len, count, blk_idx, blk_bias, partials, sb)
  switch (dm.g_q) {
    case 1: DASH_DEC(1); break;
    case 2: DASH_DEC(2); break;
    case 4: DASH_DEC(4); break;
    case 8: DASH_DEC(8); break;
    case 16: DASH_DEC(16); break;
    default: return cudaErrorInvalidValue;
  }
#undef DASH_DEC
  count_launch();
  if (e != cudaSuccess) return e;
  const long long rows = (long long)dm.batch * dm.h_q;
  e = launch_chained(decode_merge_kernel<T, D>, dim3((unsigned)((rows + 3) / 4)), dim3(128), 0, st, dm, ns,
                     (const float*)partials, (T*)O);
  count_launch();
  return e;
}

template <typename T, int D>
static cudaError_t launch_merge(const Dims& dm, int ns, const float* partials, void* O, cudaStream_t st) {
  const long long rows = (long long)dm.batch * dm.h_q;
  cudaError_t e = launch_chained(decode_merge_kernel<T, D>, dim3((unsigned)((rows + 3) / 4)), dim3(128), 0, st, dm, ns,
                                 partials, (T*)O);
  count_launch();
  return e;
}

cudaError_t launch_attend_decode_ex(const Dims& dm, const void* Q, const void* K, const void* V, const int* kv_len,
                                    const int* count, const int* blk_idx, const float* blk_bias, void* O,
                                    float* partials, StatusBlock* sb, cudaStream_t st) {
  if (decode_use_sm100(dm)) {
    // bf16, head_dim 128, chunks of 64 or 128: TMA-fed tensor-core split kernel, then the common merge
    const int ns = decode_num_splits(dm);
    // with a workspace (status block + arrival counters) the last split of each group merges in the same kernel
    const bool fused = sb != nullptr && dm.batch * dm.h_kv <= ARRIVAL_COUNTERS;
    cudaError_t e = launch_decode_sm100(dm, ns, Q, K, V, kv_len, count, blk_idx, blk_bias, partials, fused ? O : nullptr,
                                        sb, st);
    if (e != cudaSuccess || fused) return e;
    return dm.d == 128 ? launch_merge<__nv_bfloat16, 128>(dm, ns, partials, O, st)
                       : launch_merge<__nv_bfloat16, 64>(dm, ns, partials, O, st);
  }
  return launch_attend_decode(dm, Q, K, V, kv_len, count, blk_idx, blk_bias, O, partials, sb, st);
}

cudaError_t launch_attend_decode(const Dims& dm, const void* Q, const void* K, const void* V, const int* kv_len,
                                 const int* count, const int* blk_idx, const float* blk_bias, void* O,
                                 float* partials, StatusBlock* sb, cudaStream_t st) {
  if (dm.dtype == DASH_BF16) {
    if (dm.d == 128) return launch_dec<__nv_bfloat16, 128>(dm, Q, K, V, kv_len, count, blk_idx, blk_bias, O, partials, sb, st);
    return launch_dec<__nv_bfloat16, 64>(dm, Q, K, V, kv_len, count, blk_idx, blk_bias, O, partials, sb, st);
  }
  if (dm.d == 128) return launch_dec<float, 128>(dm, Q, K, V, kv_len, count, blk_idx, blk_bias, O, partials, sb, st);
  return launch_dec<float, 64>(dm, Q, K, V, kv_len, count, blk_idx, blk_bias, O, partials, sb, st);
}

}  // namespace dash

// ---------------------------------------------------------------------------------------------------
// dash_attn_attend_decode_static: the same split-KV decode attention with NO caller-provided scratch.
// The per-split partial results (m, l, O) live in the fixed device array below instead of a workspace.
// ---------------------------------------------------------------------------------------------------
namespace dash {

constexpr size_t DECODE_STATIC_MAX_FLOATS = (size_t)1 << 20;  // 4 MiB, held by every GPU that loads the library
static __device__ __align__(256) float g_decode_static_scratch[DECODE_STATIC_MAX_FLOATS];

// In host code the array's name is only a handle; the device address has to be asked for, once per device,
// with that device current.
static cudaError_t decode_static_scratch(float** out) {
  static std::mutex mu;
  static float* per_device[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (!per_device[dev]) {
    float* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_decode_static_scratch);
    if (e != cudaSuccess) return e;
    per_device[dev] = ptr;
  }
  *out = per_device[dev];
  return cudaSuccess;
}

}  // namespace dash

extern "C" int dash_attn_attend_decode_static(const dash_params* p, const void* Q, const void* Kcache,
                                              const void* Vcache, const int32_t* kv_len, const int32_t* count,
                                              const int32_t* blk_idx, const float* blk_bias, void* O, void* stream) {
  using namespace dash;
  Dims dm;
  int rc = validate_params(p, &dm);
  if (rc != DASH_OK) return rc;
  if (!dm.decode) return DASH_ERR_INVALID_ARG;
  if (!Q || !Kcache || !Vcache || !count || !O) return DASH_ERR_INVALID_ARG;
  if (dm.T_s > 0 && (!blk_idx || !blk_bias)) return DASH_ERR_INVALID_ARG;
  const uintptr_t bits = (uintptr_t)Q | (uintptr_t)Kcache | (uintptr_t)Vcache | (uintptr_t)O;
  if (bits & 15) return DASH_ERR_INVALID_ARG;
  if (decode_partial_bytes(dm) > DECODE_STATIC_MAX_FLOATS * sizeof(float)) return DASH_ERR_TOO_LARGE;
  if ((rc = validate_device()) != DASH_OK) return rc;
  float* scratch = nullptr;
  if (decode_static_scratch(&scratch) != cudaSuccess) return DASH_ERR_CUDA;
  // every partial slot that the merge kernel reads is written by the split kernel of the same call,
  // so nothing left over from an earlier call needs clearing
  return launch_attend_decode(dm, Q, Kcache, Vcache, kv_len, count, blk_idx, blk_bias, O, scratch, nullptr,
                              (cudaStream_t)stream) == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
}

