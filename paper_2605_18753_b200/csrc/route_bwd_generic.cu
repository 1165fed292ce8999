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
// Only routed chunks are touched (two sweeps over the row's list; the chunk logits are recomputed from Q and Kbar).
//
// summaries_bwd_kernel: one warp per (batch, KV head, chunk): Eq. 3, kbar_c = sum_t a_t k_t with
// a = softmax(<qbar, k_t>/sqrt(d)) (a_t = 1/B without a summary query): dk_t += a_t dkbar_c + ds_t qbar/sqrt(d),
// ds_t = a_t (<k_t, dkbar_c> - sum_u a_u <k_u, dkbar_c>), dqbar += sum_t ds_t k_t / sqrt(d).
#include "common.cuh"

namespace dash {

constexpr int RB_WARPS = 4;

template <typename T, int D>
__global__ void __launch_bounds__(RB_WARPS * 32)
route_bwd_kernel(Dims dm, const T* __restrict__ Q, const float* __restrict__ Kbar, const int* __restrict__ count,
                 const int* __restrict__ blk_idx, const float* __restrict__ tau, const float* __restrict__ dbias,
                 float* __restrict__ dQr, float* __restrict__ dKbar) {
  constexpr int VPL = D / 32;
  constexpr int MAXG = 16;
  const int lane = threadIdx.x & 31;
  const long long gw = (long long)blockIdx.x * RB_WARPS + (threadIdx.x >> 5);
  const long long total = (long long)dm.batch * dm.h_kv * dm.seq_q;
  if (gw >= total) return;
  const int i = (int)(gw % dm.seq_q);
  const int r = (int)((gw / dm.seq_q) % dm.h_kv);
  const int b = (int)(gw / ((long long)dm.seq_q * dm.h_kv));
  const int G = dm.g_q;
  const long long grp = (long long)b * dm.h_kv + r;
  // fp32 gradient of Q from the routing: [batch, seq_q, h_q, d], every row written (zeros where nothing is routed)
  float* dq_out = dQr + (((long long)b * dm.seq_q + i) * dm.h_q + (long long)r * G) * D + lane * VPL;
  const int c_own = i / dm.B;
  const int n_local = min(dm.local_blocks, c_own);              // window chunks close the list and carry no gradient
  const int n_routed = count[grp * dm.seq_q + i] - n_local;
  float q[MAXG][VPL], dq[MAXG][VPL];
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int v = 0; v < VPL; ++v) dq[h][v] = 0.f;
  if (n_routed > 0) {
    const long long loff = grp * dm.list_rows + list_row_offset(dm, i);
    const float* kb = Kbar + grp * dm.T_s * D + lane * VPL;
    float th[MAXG];
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
    // margins of one routed chunk for all heads of the group: m_h = x_scale <q_h, kbar_c> - tau_h (clamped at 0)
    auto margins = [&](int c, float* m) {
      float kv[VPL];
#pragma unroll
      for (int v = 0; v < VPL; ++v) kv[v] = kb[(long long)c * D + v];
      for (int h = 0; h < G; ++h) {
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < VPL; ++v) s = fmaf(q[h][v], kv[v], s);
        m[h] = fmaxf(warp_sum(s) * dm.x_scale - th[h], 0.f);
      }
    };
    // sweep 1: per head A_h = sum_c s_hc dw_c / g_q and S_h = sum_c s_hc
    float A[MAXG], S[MAXG];
    for (int h = 0; h < G; ++h) A[h] = S[h] = 0.f;
    for (int k = 0; k < n_routed; ++k) {
      const int c = blk_idx[loff + k];
      float m[MAXG];
      margins(c, m);
      float w = 0.f;
      for (int h = 0; h < G; ++h) w += pow_e(m[h], e_int, e);
      w /= (float)G;
      const float dw = w > 0.f ? (dbias[loff + k] - dmean) * dm.inv_sigma / w : 0.f;
      for (int h = 0; h < G; ++h) {
        const float s = pow_em1(m[h], e_int, e);
        A[h] += s * dw / (float)G;
        S[h] += s;
      }
    }
    // sweep 2: dz_hc, then dq_h and dkbar_c
    const float zscale = dm.x_scale / (1.f / e);       // gamma / sqrt(d) = x_scale / (alpha - 1)
    for (int k = 0; k < n_routed; ++k) {
      const int c = blk_idx[loff + k];
      float m[MAXG];
      margins(c, m);
      float w = 0.f;
      for (int h = 0; h < G; ++h) w += pow_e(m[h], e_int, e);
      w /= (float)G;
      const float dw = w > 0.f ? (dbias[loff + k] - dmean) * dm.inv_sigma / w : 0.f;
      float kv[VPL], dkb[VPL];
#pragma unroll
      for (int v = 0; v < VPL; ++v) { kv[v] = kb[(long long)c * D + v]; dkb[v] = 0.f; }
      for (int h = 0; h < G; ++h) {
        const float s = pow_em1(m[h], e_int, e);
        const float dz = S[h] > 0.f ? s * (dw / (float)G - A[h] / S[h]) : 0.f;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
          dq[h][v] = fmaf(dz, kv[v], dq[h][v]);
          dkb[v] = fmaf(dz, q[h][v], dkb[v]);
        }
      }
      float* dst = dKbar + (grp * dm.T_s + c) * D + lane * VPL;
#pragma unroll
      for (int v = 0; v < VPL; ++v) atomicAdd(dst + v, dkb[v] * zscale);
    }
    for (int h = 0; h < G; ++h)
#pragma unroll
      for (int v = 0; v < VPL; ++v) dq[h][v] *= zscale;
  }
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
#define DASH_RB(T, D) \
  route_bwd_kernel<T, D><<<grid, RB_WARPS * 32, 0, st>>>(dm, (const T*)Q, Kbar, count, blk_idx, tau, dbias, dQr, dKbar)
  if (dm.dtype == DASH_BF16) {
    if (dm.d == 128) DASH_RB(__nv_bfloat16, 128); else DASH_RB(__nv_bfloat16, 64);
  } else {
    if (dm.d == 128) DASH_RB(float, 128); else DASH_RB(float, 64);
  }
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
