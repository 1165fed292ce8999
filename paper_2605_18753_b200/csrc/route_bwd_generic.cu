// Backward of Stage 1 (routing) and Stage 0 (chunk summaries), prefill, CUDA-core correctness path.
//
// Section 3.5 notes that the backward pass can reuse the forward pass's bit mask because the alpha-entmax Jacobian is
// sparse; the appendix ("The alpha-entmax mapping") states that the Jacobian has a closed form where the support is
// fixed.  From Eq. 2, p_c = [(alpha-1) z_c - tau]_+^(1/(alpha-1)) with sum_c p_c = 1: on the support
// dp_c = s_c (dz_c - dtau/(alpha-1)) with s_c = p_c^(2-alpha) = margin_c^(1/(alpha-1) - 1), and sum dp = 0 fixes
// dtau, so dz = s * (dp - <s, dp> / sum(s)) and nothing outside the support receives or passes on a gradient.
//
// route_bwd_kernel: one warp per (batch, KV head, query row).  Input: the row's routed chunk list (chunk ids), the
// thresholds tau of the group's heads, and dbias (gradient w.r.t. the log-prior bias of every routed chunk, from the
// Stage-2 backward).  Chain rule of Section 3.2 / Proposition 1:
//   bias_c = (log w_c - mean_S log w)/sigma  =>  dlogw_c = (dbias_c - mean_S dbias)/sigma,  dw_c = dlogw_c / w_c
//   w_c = mean_h p_hc                        =>  dp_hc = dw_c / g_q
//   p_h = entmax(z_h), z_hc = gamma <q_h, kbar_c>/sqrt(d)   =>  dz_h by the Jacobian above
//   dq_h = gamma/sqrt(d) sum_c dz_hc kbar_c (written, fp32);   dkbar_c += gamma/sqrt(d) sum_h dz_hc q_h (atomic, fp32)
// Only routed chunks are touched (two sweeps over the row's list, four entries at a time; the chunk logits are
// recomputed from Q and Kbar).
//
// summaries_bwd_kernel: one warp per (batch, KV head, chunk): Eq. 3, kbar_c = sum_t a_t k_t with
// a = softmax(<qbar, k_t>/sqrt(d)) (a_t = 1/B without a summary query): dk_t += a_t dkbar_c + ds_t qbar/sqrt(d),
// ds_t = a_t (<k_t, dkbar_c> - sum_u a_u <k_u, dkbar_c>), dqbar += sum_t ds_t k_t / sqrt(d).
#include "common.cuh"

namespace dash {

constexpr int RB_WARPS = 4;

// Sums V values that every lane holds across the warp with the halving exchange (V - 1 + log2(32 / V) ... shuffles
// instead of 5 V): value v ends up complete in lane v * (32 / V) as x[0]; then every value is broadcast, so that all
// lanes hold all V sums (another V shuffles).  V must be a power of two <= 32.
template <int V>
__device__ __forceinline__ void warp_sum_all(float (&x)[V], int lane) {
  float y[V];
#pragma unroll
  for (int k = 0; k < V; ++k) y[k] = x[k];
#pragma unroll
  for (int width = 16, live = V; width >= 1; width >>= 1) {
    if (live > 1) {
      const bool upper = (lane & width) != 0;
      const int half = live / 2;
#pragma unroll
      for (int k = 0; k < V / 2; ++k) {
        if (k < half) {
          const float mine = upper ? y[k + half] : y[k];
          const float give = upper ? y[k] : y[k + half];
          y[k] = mine + __shfl_xor_sync(0xffffffffu, give, width);
        }
      }
      live = half;
    } else {
      y[0] += __shfl_xor_sync(0xffffffffu, y[0], width);
    }
  }
  // the lane bits were consumed from the top: value v sits in the lane whose top log2(V) bits spell v
#pragma unroll
  for (int v = 0; v < V; ++v) x[v] = __shfl_sync(0xffffffffu, y[0], v * (32 / V));
}

// G (heads per KV head) is a template parameter so that the per-head arrays live in registers; the row's routed chunks
// are taken NB at a time: their summary rows are fetched together and the NB * G dot products are reduced together.
template <typename T, int D, int G>
__global__ void __launch_bounds__(RB_WARPS * 32)
route_bwd_kernel(Dims dm, const T* __restrict__ Q, const float* __restrict__ Kbar, const int* __restrict__ count,
                 const int* __restrict__ blk_idx, const float* __restrict__ tau, const float* __restrict__ dbias,
                 float* __restrict__ dQr, float* __restrict__ dKbar) {
  constexpr int VPL = D / 32;
  constexpr int NB = G <= 8 ? 4 : 2;           // entries per batch: NB * G <= 32 values per reduction
  const int lane = threadIdx.x & 31;
  const long long gw = (long long)blockIdx.x * RB_WARPS + (threadIdx.x >> 5);
  const long long total = (long long)dm.batch * dm.h_kv * dm.seq_q;
  if (gw >= total) return;
  const int i = (int)(gw % dm.seq_q);
  const int r = (int)((gw / dm.seq_q) % dm.h_kv);
  const int b = (int)(gw / ((long long)dm.seq_q * dm.h_kv));
  const long long grp = (long long)b * dm.h_kv + r;
  // fp32 gradient of Q from the routing: [batch, seq_q, h_q, d], every row written (zeros where nothing is routed)
  float* dq_out = dQr + (((long long)b * dm.seq_q + i) * dm.h_q + (long long)r * G) * D + lane * VPL;
  const int c_own = i / dm.B;
  const int n_local = min(dm.local_blocks, c_own);              // window chunks close the list and carry no gradient
  const int n_routed = count[grp * dm.seq_q + i] - n_local;
  float q[G][VPL], dq[G][VPL];
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int v = 0; v < VPL; ++v) dq[h][v] = 0.f;
  if (n_routed > 0) {
    const long long loff = grp * dm.list_rows + list_row_offset(dm, i);
    const float* kb = Kbar + grp * dm.T_s * D + lane * VPL;
    float th[G];
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const T* qp = Q + (long long)b * dm.qs[0] + (long long)i * dm.qs[1] + (long long)(r * G + h) * dm.qs[2] + lane * VPL;
#pragma unroll
      for (int v = 0; v < VPL; ++v) q[h][v] = to_f32<T>(qp[v]);
      th[h] = tau[((long long)b * dm.h_q + r * G + h) * dm.seq_q + i];
    }
    float dmean = 0.f;
    for (int k = lane; k < n_routed; k += 32) dmean += dbias[loff + k];
    dmean = warp_sum(dmean) / (float)n_routed;
    const float e = dm.e;
    const int e_int = dm.e_int;
    // One batch: entries k0 .. k0 + NB - 1 (those beyond the list repeat the last one and are ignored by the caller).
    // kv: their summary rows; m: the margins m_h = x_scale <q_h, kbar_c> - tau_h (clamped at 0) of every entry and head;
    // dw: the gradient w.r.t. the entry's group weight.
    auto batch = [&](int k0, int (&c)[NB], float (&kv)[NB][VPL], float (&m)[NB][G], float (&dw)[NB]) {
      float db[NB];
#pragma unroll
      for (int u = 0; u < NB; ++u) {
        const int k = min(k0 + u, n_routed - 1);
        c[u] = blk_idx[loff + k];
        db[u] = dbias[loff + k];
      }
#pragma unroll
      for (int u = 0; u < NB; ++u)
#pragma unroll
        for (int v = 0; v < VPL; ++v) kv[u][v] = kb[(long long)c[u] * D + v];
      float part[NB * G];
#pragma unroll
      for (int u = 0; u < NB; ++u)
#pragma unroll
        for (int h = 0; h < G; ++h) {
          float s = 0.f;
#pragma unroll
          for (int v = 0; v < VPL; ++v) s = fmaf(q[h][v], kv[u][v], s);
          part[u * G + h] = s;
        }
      warp_sum_all<NB * G>(part, lane);
#pragma unroll
      for (int u = 0; u < NB; ++u) {
        float w = 0.f;
#pragma unroll
        for (int h = 0; h < G; ++h) {
          m[u][h] = fmaxf(part[u * G + h] * dm.x_scale - th[h], 0.f);
          w += pow_e(m[u][h], e_int, e);
        }
        w /= (float)G;
        dw[u] = w > 0.f ? (db[u] - dmean) * dm.inv_sigma / w : 0.f;
      }
    };
    // sweep 1: per head A_h = sum_c s_hc dw_c / g_q and S_h = sum_c s_hc
    float A[G], S[G];
#pragma unroll
    for (int h = 0; h < G; ++h) A[h] = S[h] = 0.f;
    for (int k0 = 0; k0 < n_routed; k0 += NB) {
      int c[NB];
      float kv[NB][VPL], m[NB][G], dw[NB];
      batch(k0, c, kv, m, dw);
#pragma unroll
      for (int u = 0; u < NB; ++u) {
        if (k0 + u < n_routed) {
#pragma unroll
          for (int h = 0; h < G; ++h) {
            const float s = pow_em1(m[u][h], e_int, e);
            A[h] += s * dw[u] / (float)G;
            S[h] += s;
          }
        }
      }
    }
    // sweep 2: dz_hc, then dq_h and dkbar_c
    const float zscale = dm.x_scale / (1.f / e);       // gamma / sqrt(d) = x_scale / (alpha - 1)
    for (int k0 = 0; k0 < n_routed; k0 += NB) {
      int c[NB];
      float kv[NB][VPL], m[NB][G], dw[NB];
      batch(k0, c, kv, m, dw);
#pragma unroll
      for (int u = 0; u < NB; ++u) {
        if (k0 + u < n_routed) {
          float dkb[VPL];
#pragma unroll
          for (int v = 0; v < VPL; ++v) dkb[v] = 0.f;
#pragma unroll
          for (int h = 0; h < G; ++h) {
            const float s = pow_em1(m[u][h], e_int, e);
            const float dz = S[h] > 0.f ? s * (dw[u] / (float)G - A[h] / S[h]) : 0.f;
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
              dq[h][v] = fmaf(dz, kv[u][v], dq[h][v]);
              dkb[v] = fmaf(dz, q[h][v], dkb[v]);
            }
          }
          float* dst = dKbar + (grp * dm.T_s + c[u]) * D + lane * VPL;
          // one vector reduction per lane (16 or 8 bytes): a quarter / half of the requests of scalar atomic adds, and
          // the requests, not the bytes, are what the L2 atomic units count
          if constexpr (VPL == 4)
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(dkb[0] * zscale), "f"(dkb[1] * zscale),
                         "f"(dkb[2] * zscale), "f"(dkb[3] * zscale) : "memory");
          else
            asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(dst), "f"(dkb[0] * zscale), "f"(dkb[1] * zscale) : "memory");
        }
      }
    }
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
      for (int v = 0; v < VPL; ++v) dq[h][v] *= zscale;
  }
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int v = 0; v < VPL; ++v) dq_out[(long long)h * D + v] = dq[h][v];
}

template <typename T, int D>
__global__ void __launch_bounds__(RB_WARPS * 32)
summaries_bwd_kernel(Dims dm, const T* __restrict__ K, const float* __restrict__ qbar, long long qbar_chunk_stride,
                     const float* __restrict__ dKbar, float* __restrict__ dK, float* __restrict__ dqbar) {
  constexpr int VPL = D / 32;
  const int lane = threadIdx.x & 31;
  const long long gw = (long long)blockIdx.x * RB_WARPS + (threadIdx.x >> 5);
  const long long total = (long long)dm.batch * dm.h_kv * dm.T_s;
  if (gw >= total) return;
  const int c = (int)(gw % dm.T_s);
  const int r = (int)((gw / dm.T_s) % dm.h_kv);
  const int b = (int)(gw / ((long long)dm.T_s * dm.h_kv));
  const T* kp = K + (long long)b * dm.ks[0] + (long long)c * dm.B * dm.ks[1] + (long long)r * dm.ks[2] + lane * VPL;
  float* dkp = dK + (((long long)b * dm.seq_kv + (long long)c * dm.B) * dm.h_kv + r) * D + lane * VPL;
  const long long gtok = (long long)dm.h_kv * D;
  float g[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) g[v] = dKbar[(((long long)b * dm.h_kv + r) * dm.T_s + c) * D + lane * VPL + v];
  if (qbar == nullptr) {
    const float inv = 1.f / (float)dm.B;
    for (int t = 0; t < dm.B; ++t)
#pragma unroll
      for (int v = 0; v < VPL; ++v) dkp[(long long)t * gtok + v] += g[v] * inv;
    return;
  }
  float qv[VPL];
  const float* qp = qbar + (long long)c * qbar_chunk_stride + (long long)r * D + lane * VPL;
#pragma unroll
  for (int v = 0; v < VPL; ++v) qv[v] = qp[v];
  // pass 1: softmax statistics of s_t = <qbar, k_t>/sqrt(d) and sum_t a_t <k_t, g>
  float mx = -INFINITY;
  for (int t = 0; t < dm.B; ++t) {
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < VPL; ++v) s = fmaf(qv[v], to_f32<T>(kp[(long long)t * dm.ks[1] + v]), s);
    mx = fmaxf(mx, warp_sum(s) * dm.sm_scale);
  }
  float l = 0.f, ada = 0.f;
  for (int t = 0; t < dm.B; ++t) {
    float s = 0.f, da = 0.f;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      const float kvv = to_f32<T>(kp[(long long)t * dm.ks[1] + v]);
      s = fmaf(qv[v], kvv, s);
      da = fmaf(g[v], kvv, da);
    }
    const float p = __expf(warp_sum(s) * dm.sm_scale - mx);
    l += p;
    ada += p * warp_sum(da);
  }
  ada /= l;
  // pass 2: dk_t and dqbar
  float dqb[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) dqb[v] = 0.f;
  for (int t = 0; t < dm.B; ++t) {
    float kvv[VPL], s = 0.f, da = 0.f;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      kvv[v] = to_f32<T>(kp[(long long)t * dm.ks[1] + v]);
      s = fmaf(qv[v], kvv[v], s);
      da = fmaf(g[v], kvv[v], da);
    }
    const float a = __expf(warp_sum(s) * dm.sm_scale - mx) / l;
    const float dst = a * (warp_sum(da) - ada);
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      dkp[(long long)t * gtok + v] += a * g[v] + dst * qv[v] * dm.sm_scale;
      dqb[v] = fmaf(dst, kvv[v], dqb[v]);
    }
  }
  if (dqbar) {
    float* dq = dqbar + (long long)c * qbar_chunk_stride + (long long)r * D + lane * VPL;
#pragma unroll
    for (int v = 0; v < VPL; ++v) atomicAdd(dq + v, dqb[v] * dm.sm_scale);
  }
}

cudaError_t launch_route_bwd(const Dims& dm, const void* Q, const float* Kbar, const int* count, const int* blk_idx,
                             const float* tau, const float* dbias, float* dQr, float* dKbar, cudaStream_t st) {
  const size_t kb_bytes = (size_t)dm.batch * dm.h_kv * (size_t)dm.T_s * dm.d * sizeof(float);
  if (kb_bytes > 0) {
    cudaError_t e = cudaMemsetAsync(dKbar, 0, kb_bytes, st);
    if (e != cudaSuccess) return e;
  }
  const long long total = (long long)dm.batch * dm.h_kv * dm.seq_q;
  const unsigned grid = (unsigned)((total + RB_WARPS - 1) / RB_WARPS);
#define DASH_RB(T, D, GV) \
  route_bwd_kernel<T, D, GV><<<grid, RB_WARPS * 32, 0, st>>>(dm, (const T*)Q, Kbar, count, blk_idx, tau, dbias, dQr, dKbar)
#define DASH_RB_G(T, D)                   \
  switch (dm.g_q) {                       \
    case 1: DASH_RB(T, D, 1); break;      \
    case 2: DASH_RB(T, D, 2); break;      \
    case 4: DASH_RB(T, D, 4); break;      \
    case 8: DASH_RB(T, D, 8); break;      \
    case 16: DASH_RB(T, D, 16); break;    \
    default: return cudaErrorInvalidValue; \
  }
  if (dm.dtype == DASH_BF16) {
    if (dm.d == 128) { DASH_RB_G(__nv_bfloat16, 128) } else { DASH_RB_G(__nv_bfloat16, 64) }
  } else {
    if (dm.d == 128) { DASH_RB_G(float, 128) } else { DASH_RB_G(float, 64) }
  }
#undef DASH_RB_G
#undef DASH_RB
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_summaries_bwd(const Dims& dm, const void* K, const float* qbar, long long qbar_chunk_stride,
                                 const float* dKbar, float* dK, float* dqbar, size_t dqbar_bytes, cudaStream_t st) {
  if (dqbar && dqbar_bytes > 0) {
    cudaError_t e = cudaMemsetAsync(dqbar, 0, dqbar_bytes, st);
    if (e != cudaSuccess) return e;
  }
  const long long total = (long long)dm.batch * dm.h_kv * dm.T_s;
  if (total == 0) return cudaSuccess;
  const unsigned grid = (unsigned)((total + RB_WARPS - 1) / RB_WARPS);
#define DASH_SB(T, D) \
  summaries_bwd_kernel<T, D><<<grid, RB_WARPS * 32, 0, st>>>(dm, (const T*)K, qbar, qbar_chunk_stride, dKbar, dK, dqbar)
  if (dm.dtype == DASH_BF16) {
    if (dm.d == 128) DASH_SB(__nv_bfloat16, 128); else DASH_SB(__nv_bfloat16, 64);
  } else {
    if (dm.d == 128) DASH_SB(float, 128); else DASH_SB(float, 64);
  }
#undef DASH_SB
  count_launch();
  return cudaGetLastError();
}

}  // namespace dash
