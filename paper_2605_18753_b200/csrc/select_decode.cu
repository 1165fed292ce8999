// Stage 1 for decode (Eq. 2, Eq. 4, Algorithm 2, Proposition 1): one query row per sequence.
//
// Decode routing is HBM-bound on the summary cache (every candidate's kbar row is read once per step and
// per KV head), so it is split in two kernels:
//   decode_scores_kernel  many thread blocks per (batch, KV head) stream kbar with fully coalesced 512-byte
//                         row reads (one warp per row, four rows in flight per warp) and write the scaled
//                         chunk logits x = gamma(alpha-1) <q, kbar_c>/sqrt(d) of the g_q heads to a small
//                         fp32 scratch (b * h_q * T_s floats, stays in L2);
//   decode_route_kernel   one thread block of 16 warps per (batch, KV head) loads its g_q logit rows into shared
//                         memory, finds tau per head (Newton; one warp per head with its share of the row in
//                         registers, no barrier inside the iteration), then forms the group weights, mask words, log w,
//                         mu and the compact (chunk, bias) list.
// With a local window of L chunks the last L chunks before the own one are not scored; the routing kernel sets
// their bits and appends them to the list with bias 0.
#include <type_traits>

#include "common.cuh"

namespace dash {

namespace {

constexpr int SC_WARPS = 8;
constexpr int SC_ROWS_PER_BLOCK = 256;   // summary rows one thread block scores
constexpr int RT_THREADS = 512;      // 128 registers per thread: a Newton warp keeps 64 logits per lane in registers
constexpr int RT_LOADS = 4;           // logits per head a thread requests per sweep (2048 candidates: one sweep)
constexpr int RT_MAX_NEWTON = 64, RT_MAX_NEWTON_GENERIC = 400;

// Sum V values held by every lane across the warp with V-1+... shuffles (halving exchange): after the
// call lane 0..V-1 ... we only need the totals in ONE lane per value, so the classic butterfly that halves
// the number of live values per step is used; value v ends up (fully reduced) in lane (v * 32 / V) for V | 32.
template <int V>
__device__ __forceinline__ void warp_reduce_many(float (&x)[V], int lane) {
#pragma unroll
  for (int width = 16, live = V; width >= 1; width >>= 1) {
    if (live > 1) {
      // exchange halves: lanes with bit `width` clear keep the lower half of the live values, others the upper
      const bool upper = (lane & width) != 0;
      const int half = live / 2;
#pragma unroll
      for (int k = 0; k < V / 2; ++k) {
        if (k < half) {
          const float mine = upper ? x[k + half] : x[k];
          const float give = upper ? x[k] : x[k + half];
          x[k] = mine + __shfl_xor_sync(0xffffffffu, give, width);
        }
      }
      live = half;
    } else {
      x[0] += __shfl_xor_sync(0xffffffffu, x[0], width);
    }
  }
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(SC_WARPS * 32)
decode_scores_kernel(Dims dm, const T* __restrict__ Q, const float* __restrict__ Kbar, const int* __restrict__ kv_len,
                     float* __restrict__ xs) {
  constexpr int VPL = D / 32;   // floats per lane of one summary row
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int r = blockIdx.y, b = blockIdx.z;
  int L = kv_len ? kv_len[b] : dm.seq_kv;     // the caller's input, not a product of the chain: read it before the wait
  chain_wait();
  chain_release();
  L = max(1, min(L, dm.seq_kv));
  const int n_cand = max(min((L - 1) / dm.B, dm.T_s) - dm.local_blocks, 0);   // window chunks are not scored
  const int c_begin = blockIdx.x * SC_ROWS_PER_BLOCK;
  const int c_end = min(n_cand, c_begin + SC_ROWS_PER_BLOCK);
  if (c_begin >= c_end) return;

  float q[G][VPL];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const T* qp = Q + (long long)b * dm.qs[0] + (long long)(r * G + g) * dm.qs[2] + lane * VPL;
#pragma unroll
    for (int v = 0; v < VPL; ++v) q[g][v] = to_f32<T>(qp[v]) * dm.x_scale;
  }
  const float* kb = Kbar + ((long long)b * dm.h_kv + r) * dm.T_s * D + lane * VPL;
  float* xo = xs + ((long long)b * dm.h_kv + r) * G * dm.T_s;

  constexpr int RB = (G <= 8) ? 4 : 2;        // rows per iteration: RB * G values reduced together (<= 32)
  for (int c0 = c_begin + warp * RB; c0 < c_end; c0 += SC_WARPS * RB) {
    float kv[RB][VPL];
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      const int c = min(c0 + u, c_end - 1);
      if constexpr (VPL == 4) {
        const float4 f = __ldcs(reinterpret_cast<const float4*>(kb + (long long)c * D));   // read once: streaming
        kv[u][0] = f.x; kv[u][1] = f.y; kv[u][2] = f.z; kv[u][3] = f.w;
      } else {
        const float2 f = __ldcs(reinterpret_cast<const float2*>(kb + (long long)c * D));
        kv[u][0] = f.x; kv[u][1] = f.y;
      }
    }
    float part[RB * G];
#pragma unroll
    for (int u = 0; u < RB; ++u)
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < VPL; ++v) s = fmaf(q[g][v], kv[u][v], s);
        part[u * G + g] = s;
      }
    warp_reduce_many<RB * G>(part, lane);
    // value v = u*G + g is complete in lane v * (32 / (RB*G)) as part[0]
    constexpr int STRIDE = 32 / (RB * G);
    if (lane % STRIDE == 0) {
      const int v = lane / STRIDE, u = v / G, g = v % G;
      if (c0 + u < c_end) xo[(long long)g * dm.T_s + c0 + u] = part[0];
    }
  }
}

// Row pitch of the logits in decode_route_kernel's shared memory (host and device agree through this helper).
__host__ __device__ inline int route_stride(int n) { return ((n + 31) / 32) * 32 + 32; }

template <int G>
__global__ void __launch_bounds__(RT_THREADS)
decode_route_kernel(Dims dm, const float* __restrict__ xs, const int* __restrict__ kv_len, uint32_t* __restrict__ mask,
                    int* __restrict__ count, int* __restrict__ blk_idx, float* __restrict__ blk_bias,
                    float* __restrict__ tau_out) {
  extern __shared__ __align__(16) float sm[];
  constexpr int NW = RT_THREADS / 32;
  static_assert(NW <= 32 && G <= NW, "a lane per warp in the reduction of the maxima; a warp per head in the iteration");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = blockIdx.x, b = blockIdx.y;
  int L = kv_len ? kv_len[b] : dm.seq_kv;     // the caller's input, not a product of the chain: read it before the wait
  chain_wait();
  chain_release();
  L = max(1, min(L, dm.seq_kv));
  const int c_own = (L - 1) / dm.B;
  const int n_vis = min(c_own, dm.T_s);                 // chunks before the own one: candidates, then the window
  const int n_cand = max(n_vis - dm.local_blocks, 0);   // scored by entmax
  const int stride = route_stride(n_vis);
  float* X = sm;                                 // [G][stride] all logits of the group
  float* taus = X + (size_t)G * stride;          // [G] (32 floats reserved)
  float* wsum = taus + 32;                       // per-word sum of log w   [W]
  int* wcnt = reinterpret_cast<int*>(wsum + dm.W);   // per-word popcount / exclusive prefix [W + 1]
  float* red = reinterpret_cast<float*>(wcnt + dm.W + 1);   // [NW][G] per-warp maxima
  const long long grp = (long long)b * dm.h_kv + r;
  const float* xg = xs + grp * G * dm.T_s;

  // ---- logits -> shared memory, row maxima
  float mx[G];
#pragma unroll
  for (int g = 0; g < G; ++g) mx[g] = -INFINITY;
  // all of a thread's loads of one sweep are issued before the first is used (one L2 round trip per sweep)
  for (int c0 = 0; c0 < n_cand; c0 += RT_LOADS * RT_THREADS) {
    float v[G][RT_LOADS];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int u = 0; u < RT_LOADS; ++u) {
        const int c = c0 + u * RT_THREADS + tid;
        v[g][u] = c < n_cand ? __ldcg(xg + (long long)g * dm.T_s + c) : -INFINITY;
      }
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int u = 0; u < RT_LOADS; ++u) {
        const int c = c0 + u * RT_THREADS + tid;
        if (c < n_cand) X[(size_t)g * stride + c] = v[g][u];
        mx[g] = fmaxf(mx[g], v[g][u]);
      }
  }
  // maxima through the integer warp reduction (one instruction instead of five shuffles): floats map to
  // signed integers of the same order by flipping the magnitude bits of the negative ones
  auto f2ord = [](float f) { const int i = __float_as_int(f); return i ^ ((i >> 31) & 0x7fffffff); };
  auto ord2f = [](int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); };
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const int m = __reduce_max_sync(0xffffffffu, f2ord(mx[g]));
    if (lane == 0) red[warp * G + g] = ord2f(m);
  }
  __syncthreads();
#pragma unroll
  for (int g = 0; g < G; ++g) mx[g] = ord2f(__reduce_max_sync(0xffffffffu, f2ord(lane < NW ? red[lane * G + g] : -INFINITY)));

  // ---- tau per head.  One warp per head, no barrier inside the iteration: a lane keeps its share of the row (up to
  // 64 logits, i.e. rows of up to 2048 candidates; anything beyond is re-read from shared memory) in registers over all
  // passes, a pass is the lane's sums, two warp sums and the step.  The start is the larger of the all-active root and
  // the normal-tail estimate from the row's mean and variance (closed forms for alpha = 2 and 1.5, as in the prefill
  // kernel); either side of the root is a valid start: from the left the iterates rise monotonically, from the right
  // one step lands on the left.
  const int e_int = dm.e_int;
  const float e = dm.e;
  if (warp < G) {
    const int g = warp;
    float tau = 0.f;
    if (n_cand > 0) {
      const float* x = X + (size_t)g * stride;
      float mxg = 0.f;
#pragma unroll
      for (int k = 0; k < G; ++k) if (k == g) mxg = mx[k];
      constexpr int RPL = 64;                       // logits a lane holds
      float xr[RPL];
#pragma unroll
      for (int u = 0; u < RPL; ++u) {
        const int c = lane + 32 * u;
        xr[u] = c < n_cand ? x[c] : -INFINITY;
      }
      // moments about the maximum
      float s1 = 0.f, s2 = 0.f;
#pragma unroll
      for (int u = 0; u < RPL; ++u) {
        const float y = xr[u] > -INFINITY ? xr[u] - mxg : 0.f;
        s1 += y;
        s2 = fmaf(y, y, s2);
      }
      for (int c = lane + 32 * RPL; c < n_cand; c += 32) {
        const float y = x[c] - mxg;
        s1 += y;
        s2 = fmaf(y, y, s2);
      }
      s1 = warp_sum(s1);
      s2 = warp_sum(s2);
      {
        const float n = (float)n_cand;
        float t = -1.f;
        if (e_int == 1) {
          t = (s1 - 1.f) / n;
        } else if (e_int == 2) {
          const float mean = s1 / n, ss = s2 - s1 * mean;
          if (ss < 1.f) t = mean - sqrtf((1.f - ss) / n);
          if (n_cand >= 8 && ss > 0.f) {
            const float L = -__logf(fminf(fmaxf(ss, 0.3334f), 1e7f));
            const float z = fmaf(fmaf(fmaf(fmaf(-8.93074e-05f, L, -0.0037117f), L, -0.0612527f), L, -0.717421f), L, -0.499476f);
            t = fmaxf(t, fmaf(z, sqrtf(ss / n), mean));
          }
        }
        tau = mxg + fminf(fmaxf(t, -1.f), -1e-6f);
      }
      auto newton = [&](auto ei_tag) {
        constexpr int EI = decltype(ei_tag)::value;
        const int max_it = EI ? RT_MAX_NEWTON : RT_MAX_NEWTON_GENERIC;
        for (int it = 0; it < max_it; ++it) {
          float F[4] = {0.f, 0.f, 0.f, 0.f}, Gs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int u = 0; u < RPL; ++u) {
            const float m = fmaxf(xr[u] - tau, 0.f);
            F[u & 3] += pow_e(m, EI, e);
            Gs[u & 3] += pow_em1(m, EI, e);
          }
          for (int c = lane + 32 * RPL; c < n_cand; c += 32) {
            const float m = fmaxf(x[c] - tau, 0.f);
            F[0] += pow_e(m, EI, e);
            Gs[0] += pow_em1(m, EI, e);
          }
          const float f = warp_sum((F[0] + F[1]) + (F[2] + F[3]));
          const float gs = warp_sum((Gs[0] + Gs[1]) + (Gs[2] + Gs[3]));
          if (fabsf(f - 1.f) <= NEWTON_F_TOL || !(gs > 0.f)) break;
          const float nt = tau + newton_delta(f, gs, EI, e);
          if (nt == tau) break;
          tau = nt;
        }
      };
      switch (e_int) {
        case 1: newton(std::integral_constant<int, 1>{}); break;
        case 2: newton(std::integral_constant<int, 2>{}); break;
        case 4: newton(std::integral_constant<int, 4>{}); break;
        default: newton(std::integral_constant<int, 0>{}); break;
      }
    }
    if (lane == 0) {
      taus[g] = tau;
      if (tau_out) tau_out[(long long)b * dm.h_q + r * G + g] = tau;
    }
  }
  __syncthreads();

  // pass 1: one warp per 32-chunk mask word: support bits, log w (stashed over head 0's logits)
  const float log_gq = logf((float)G);
  uint32_t* mrow = mask + grp * dm.W;
  for (int j = warp; j < dm.W; j += RT_THREADS / 32) {
    const int c = j * 32 + lane;
    bool sel = false;
    float lw = INFINITY;
    if (c < n_cand) {
      float mstar = 0.f;
      for (int g = 0; g < G; ++g) mstar = fmaxf(mstar, X[(size_t)g * stride + c] - taus[g]);
      if (mstar > 0.f) {
        sel = true;
        const float inv = 1.f / mstar;
        float s = 0.f;
        for (int g = 0; g < G; ++g) s += pow_e(fmaxf(X[(size_t)g * stride + c] - taus[g], 0.f) * inv, e_int, e);
        lw = e * logf(mstar) + logf(s) - log_gq;
      }
    }
    const float ls = warp_sum(sel ? lw : 0.f);
    if (c >= n_cand && c < n_vis) {                 // window chunk: listed with bias 0, outside mu
      sel = true;
      lw = -INFINITY;
    }
    const uint32_t word = __ballot_sync(0xffffffffu, sel);
    if (c < n_vis) X[c] = lw;                       // +inf marks "not routed", -inf a window chunk
    if (lane == 0) {
      mrow[j] = word | (((c_own >> 5) == j) ? (1u << (c_own & 31)) : 0u);
      wsum[j] = ls;
      wcnt[j] = __popc(word);
    }
  }
  __syncthreads();
  // exclusive prefix of the per-word counts and the total of log w (W <= a few hundred: one warp)
  if (warp == 0) {
    int base = 0;
    float tot = 0.f;
    for (int j0 = 0; j0 < dm.W; j0 += 32) {
      const int j = j0 + lane;
      const int v = j < dm.W ? wcnt[j] : 0;
      const float sv = j < dm.W ? wsum[j] : 0.f;
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      if (j < dm.W) wcnt[j] = base + incl - v;
      base += __shfl_sync(0xffffffffu, incl, 31);
      tot += warp_sum(sv);
    }
    if (lane == 0) {
      wcnt[dm.W] = base;
      wsum[0] = tot;
      count[grp] = base;
    }
  }
  __syncthreads();
  const int nlist = wcnt[dm.W];                  // routed + window chunks
  const int nsel = nlist - (n_vis - n_cand);     // routed only: the denominator of mu
  if (nlist > 0) {
    const float mu = nsel > 0 ? wsum[0] / (float)nsel : 0.f;
    const long long loff = grp * dm.list_rows;
    for (int j = warp; j * 32 < n_vis; j += RT_THREADS / 32) {
      const int c = j * 32 + lane;
      const float lw = (c < n_vis) ? X[c] : INFINITY;
      const bool sel = lw < INFINITY;
      const uint32_t word = __ballot_sync(0xffffffffu, sel);
      if (sel) {
        const long long pos = loff + wcnt[j] + __popc(word & ((1u << lane) - 1u));
        blk_bias[pos] = lw == -INFINITY ? 0.f : (lw - mu) * dm.inv_sigma;
        if (blk_idx) blk_idx[pos] = c;
      }
    }
  }
}

}  // namespace

size_t select_decode_scratch_bytes(const Dims& dm) {
  return dm.decode ? (size_t)dm.batch * dm.h_q * (size_t)(dm.T_s > 0 ? dm.T_s : 1) * sizeof(float) : 0;
}

static size_t route_smem(const Dims& dm) {
  // logits, taus, per-word sums and counts, per-warp maxima
  return ((size_t)dm.g_q * route_stride(dm.T_s) + 32 + dm.W + dm.W + 1 + 8 +
          (size_t)(RT_THREADS / 32) * dm.g_q) * sizeof(float);
}

bool select_decode_supported(const Dims& dm) { return dm.decode && route_smem(dm) <= 200 * 1024; }

cudaError_t launch_select_decode(const Dims& dm, const void* Q, const float* Kbar, const int* kv_len, uint32_t* mask,
                                 int* count, int* blk_idx, float* blk_bias, float* tau, float* scratch,
                                 cudaStream_t st) {
  const int blocks_x = (dm.T_s + SC_ROWS_PER_BLOCK - 1) / SC_ROWS_PER_BLOCK;
  if (blocks_x > 0) {
    dim3 grid(blocks_x, dm.h_kv, dm.batch);
    cudaError_t le = cudaSuccess;
#define DASH_SC(T, D, G) \
  le = launch_chained(decode_scores_kernel<T, D, G>, grid, dim3(SC_WARPS * 32), 0, st, dm, (const T*)Q, Kbar, kv_len, scratch)
#define DASH_SC_G(T, D)                                \
  switch (dm.g_q) {                                    \
    case 1: DASH_SC(T, D, 1); break;                   \
    case 2: DASH_SC(T, D, 2); break;                   \
    case 4: DASH_SC(T, D, 4); break;                   \
    case 8: DASH_SC(T, D, 8); break;                   \
    case 16: DASH_SC(T, D, 16); break;                 \
    default: return cudaErrorInvalidValue;             \
  }
    if (dm.dtype == DASH_BF16) {
      if (dm.d == 128) { DASH_SC_G(__nv_bfloat16, 128) } else { DASH_SC_G(__nv_bfloat16, 64) }
    } else {
      if (dm.d == 128) { DASH_SC_G(float, 128) } else { DASH_SC_G(float, 64) }
    }
#undef DASH_SC_G
#undef DASH_SC
    count_launch();
    if (le != cudaSuccess) return le;
  }
  const size_t smem = route_smem(dm);
  cudaError_t re = cudaSuccess;
#define DASH_RT(G)                                                                                                  \
  {                                                                                                                 \
    static std::atomic<unsigned long long> configured{0};                                                           \
    cudaError_t e = allow_dynamic_smem(decode_route_kernel<G>, 200 * 1024, configured);                             \
    if (e != cudaSuccess) return e;                                                                                 \
    re = launch_chained(decode_route_kernel<G>, dim3(dm.h_kv, dm.batch), dim3(RT_THREADS), smem, st, dm,           \
                        (const float*)scratch, kv_len, mask, count, blk_idx, blk_bias, tau);                       \
  }
  switch (dm.g_q) {
    case 1: DASH_RT(1) break;
    case 2: DASH_RT(2) break;
    case 4: DASH_RT(4) break;
    case 8: DASH_RT(8) break;
    case 16: DASH_RT(16) break;
    default: return cudaErrorInvalidValue;
  }
#undef DASH_RT
  count_launch();
  return re;
}

}  // namespace dash
