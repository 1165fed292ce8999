// Backward of Stage 2, prefill, CUDA-core correctness path: gradients of the prior-biased softmax attention (Eq. 7 in
// the form of Proposition 1) with the routing held fixed.  It reuses the forward pass's bit mask and bias lists, as
// Section 3.5 notes the backward pass can (the alpha-entmax Jacobian is zero outside the support, so nothing outside
// the mask ever receives a gradient).
//
// With l_j = <q, k_j>/sqrt(d) + bias_c(j) (bias 0 and the causal mask on the own chunk), P = softmax(l), o = P V and
// an incoming dO:   dP_j = <do, v_j>,   delta = <o, do>,   dl_j = P_j (dP_j - delta),
//   dq = sum_j dl_j k_j / sqrt(d),   dk_j += dl_j q / sqrt(d),   dv_j += P_j do,
//   dbias_c += sum over the tokens of chunk c and the heads of the group of dl_j   (what the routing backward takes on).
//
// One warp per (batch, query token, query head), two sweeps over the row's chunks in the order of the forward kernel:
// the first recomputes the softmax statistics and o (so delta does not inherit the rounding of a stored bf16 output),
// the second forms dl and scatters.  Lanes own keys for the logits and head_dim slices for the accumulators; dK, dV
// and dbias are fp32 and accumulated with atomic adds (several rows and heads meet in one key), so their low bits
// depend on scheduling.
#include "common.cuh"

namespace dash {

constexpr int AB_WARPS = 4;

template <typename T, int D>
__global__ void __launch_bounds__(AB_WARPS * 32)
attend_prefill_bwd_generic_kernel(Dims dm, const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                                  const T* __restrict__ dO, const uint32_t* __restrict__ mask,
                                  const float* __restrict__ blk_bias, T* __restrict__ dQ, float* __restrict__ dK,
                                  float* __restrict__ dV, float* __restrict__ dbias) {
  constexpr int VPL = D / 32;
  __shared__ __align__(16) float qs[AB_WARPS][D];    // q / sqrt(d)
  __shared__ __align__(16) float gs[AB_WARPS][D];    // dO row
  __shared__ float ps[AB_WARPS][32], ds[AB_WARPS][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long gw = (long long)blockIdx.x * AB_WARPS + warp;
  const long long total = (long long)dm.batch * dm.seq_q * dm.h_q;
  if (gw >= total) return;
  const int h = (int)(gw % dm.h_q);
  const int i = dm.seq_q - 1 - (int)((gw / dm.h_q) % dm.seq_q);  // long rows first
  const int b = (int)(gw / ((long long)dm.h_q * dm.seq_q));
  const int r = h / dm.g_q;
  const int c_own = dm.causal ? i / dm.B : dm.T_s;

  const T* qp = Q + (long long)b * dm.qs[0] + (long long)i * dm.qs[1] + (long long)h * dm.qs[2];
  const T* gp = dO + (long long)b * dm.os[0] + (long long)i * dm.os[1] + (long long)h * dm.os[2];
  for (int k = lane; k < D; k += 32) {
    qs[warp][k] = to_f32<T>(qp[k]) * dm.sm_scale;
    gs[warp][k] = to_f32<T>(gp[k]);
  }
  __syncwarp();

  const T* kbase = K + (long long)b * dm.ks[0] + (long long)r * dm.ks[2];
  const T* vbase = V + (long long)b * dm.vs[0] + (long long)r * dm.vs[2];
  const uint32_t* mrow = mask + (((long long)b * dm.h_kv + r) * dm.seq_q + i) * dm.W;
  const long long list0 = ((long long)b * dm.h_kv + r) * dm.list_rows + list_row_offset(dm, i);
  const float* brow = blk_bias + list0;
  float* dbrow = dbias + list0;
  // gradient buffers are [batch, seq_kv, h_kv, d] fp32, contiguous
  float* dkbase = dK + (((long long)b * dm.seq_kv) * dm.h_kv + r) * D;
  float* dvbase = dV + (((long long)b * dm.seq_kv) * dm.h_kv + r) * D;
  const long long gtok = (long long)dm.h_kv * D;     // token pitch of the gradient buffers

  // logit of the lane's key in a 32-key slice (or -inf beyond the slice's end)
  auto logit = [&](int t, int t_end, float bias) -> float {
    if (t >= t_end) return -INFINITY;
    const T* kp = kbase + (long long)t * dm.ks[1];
    float a = 0.f;
#pragma unroll 4
    for (int k = 0; k < D; k += 4) {
      const float4 kv = load4(kp + k);
      const float4 qv = *reinterpret_cast<const float4*>(&qs[warp][k]);
      a = fmaf(qv.x, kv.x, a); a = fmaf(qv.y, kv.y, a); a = fmaf(qv.z, kv.z, a); a = fmaf(qv.w, kv.w, a);
    }
    return a + bias;
  };

  // ---- sweep 1: row maximum, normaliser and o (Algorithm 3 steps 8-11), then delta = <o, dO>
  float m = -INFINITY, l = 0.f, acc[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) acc[v] = 0.f;
  int cursor = 0;
  for (int j = 0; j < dm.W; ++j) {
    uint32_t word = mrow[j];
    while (word) {
      const int bit = __ffs(word) - 1;
      word &= word - 1;
      const int c = j * 32 + bit;
      if (c > c_own) continue;
      const float bias = (c == c_own) ? 0.f : brow[cursor];
      if (c != c_own) ++cursor;
      const int t_end = (c == c_own && dm.causal) ? (i + 1) : min((c + 1) * dm.B, dm.seq_kv);
      for (int t0 = c * dm.B; t0 < t_end; t0 += 32) {
        const float s = logit(t0 + lane, t_end, bias);
        const float mt = fmaxf(m, warp_max(s));
        const float corr = __expf(m - mt);
        const float p = (t0 + lane < t_end) ? __expf(s - mt) : 0.f;
        l = l * corr + warp_sum(p);
#pragma unroll
        for (int v = 0; v < VPL; ++v) acc[v] *= corr;
        ps[warp][lane] = p;
        __syncwarp();
        const int nt = min(32, t_end - t0);
        for (int u = 0; u < nt; ++u) {
          const float pu = ps[warp][u];
          const T* vp = vbase + (long long)(t0 + u) * dm.vs[1] + lane * VPL;
#pragma unroll
          for (int v = 0; v < VPL; ++v) acc[v] = fmaf(pu, to_f32<T>(vp[v]), acc[v]);
        }
        __syncwarp();
        m = mt;
      }
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  float dpart = 0.f;
#pragma unroll
  for (int v = 0; v < VPL; ++v) dpart = fmaf(acc[v] * inv, gs[warp][lane * VPL + v], dpart);
  const float delta = warp_sum(dpart);

  // ---- sweep 2: dl per key, then dq (kept), dk, dv, dbias (scattered)
  float dq[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) dq[v] = 0.f;
  cursor = 0;
  for (int j = 0; j < dm.W; ++j) {
    uint32_t word = mrow[j];
    while (word) {
      const int bit = __ffs(word) - 1;
      word &= word - 1;
      const int c = j * 32 + bit;
      if (c > c_own) continue;
      const bool routed = c != c_own;
      const float bias = routed ? brow[cursor] : 0.f;
      const int t_end = (c == c_own && dm.causal) ? (i + 1) : min((c + 1) * dm.B, dm.seq_kv);
      float dsum = 0.f;
      for (int t0 = c * dm.B; t0 < t_end; t0 += 32) {
        const int t = t0 + lane;
        const float s = logit(t, t_end, bias);
        float p = 0.f, dl = 0.f;
        if (t < t_end) {
          p = __expf(s - m) * inv;
          const T* vp = vbase + (long long)t * dm.vs[1];
          float dp = 0.f;
#pragma unroll 4
          for (int k = 0; k < D; k += 4) {
            const float4 vv = load4(vp + k);
            const float4 gv = *reinterpret_cast<const float4*>(&gs[warp][k]);
            dp = fmaf(gv.x, vv.x, dp); dp = fmaf(gv.y, vv.y, dp); dp = fmaf(gv.z, vv.z, dp); dp = fmaf(gv.w, vv.w, dp);
          }
          dl = p * (dp - delta);
        }
        dsum += dl;
        ps[warp][lane] = p;
        ds[warp][lane] = dl;
        __syncwarp();
        const int nt = min(32, t_end - t0);
        for (int u = 0; u < nt; ++u) {
          const float pu = ps[warp][u], du = ds[warp][u];
          const T* kp = kbase + (long long)(t0 + u) * dm.ks[1] + lane * VPL;
          float* dkp = dkbase + (long long)(t0 + u) * gtok + lane * VPL;
          float* dvp = dvbase + (long long)(t0 + u) * gtok + lane * VPL;
          float ak[VPL], av[VPL];
#pragma unroll
          for (int v = 0; v < VPL; ++v) {
            dq[v] = fmaf(du, to_f32<T>(kp[v]), dq[v]);
            ak[v] = du * qs[warp][lane * VPL + v];          // qs already carries 1/sqrt(d)
            av[v] = pu * gs[warp][lane * VPL + v];
          }
          // one vector reduction per lane and tensor: the L2 atomic units count requests, not bytes
          if constexpr (VPL == 4) {
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dkp), "f"(ak[0]), "f"(ak[1]), "f"(ak[2]), "f"(ak[3]) : "memory");
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dvp), "f"(av[0]), "f"(av[1]), "f"(av[2]), "f"(av[3]) : "memory");
          } else {
            asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(dkp), "f"(ak[0]), "f"(ak[1]) : "memory");
            asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(dvp), "f"(av[0]), "f"(av[1]) : "memory");
          }
        }
        __syncwarp();
      }
      if (routed) {
        const float tot = warp_sum(dsum);
        if (lane == 0) atomicAdd(dbrow + cursor, tot);
        ++cursor;
      }
    }
  }
  T* dqp = dQ + (long long)b * dm.qs[0] + (long long)i * dm.qs[1] + (long long)h * dm.qs[2] + lane * VPL;
#pragma unroll
  for (int v = 0; v < VPL; ++v) dqp[v] = from_f32<T>(dq[v] * dm.sm_scale);
}

cudaError_t launch_attend_prefill_bwd_generic(const Dims& dm, const void* Q, const void* K, const void* V,
                                              const void* dO, const uint32_t* mask, const float* blk_bias, void* dQ,
                                              float* dK, float* dV, float* dbias, cudaStream_t st) {
  // the scattered outputs start from zero
  const size_t kv_bytes = (size_t)dm.batch * dm.seq_kv * dm.h_kv * dm.d * sizeof(float);
  cudaError_t e = cudaMemsetAsync(dK, 0, kv_bytes, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(dV, 0, kv_bytes, st);
  const size_t list_bytes = (size_t)dm.batch * dm.h_kv * (size_t)dm.list_rows * sizeof(float);
  if (e == cudaSuccess && list_bytes > 0) e = cudaMemsetAsync(dbias, 0, list_bytes, st);
  if (e != cudaSuccess) return e;
  const long long total = (long long)dm.batch * dm.seq_q * dm.h_q;
  const unsigned grid = (unsigned)((total + AB_WARPS - 1) / AB_WARPS);
#define DASH_LAUNCH_AB(T, D)                                                                                     \
  attend_prefill_bwd_generic_kernel<T, D><<<grid, AB_WARPS * 32, 0, st>>>(dm, (const T*)Q, (const T*)K, (const T*)V, \
                                                                          (const T*)dO, mask, blk_bias, (T*)dQ, dK, dV, dbias)
  if (dm.dtype == DASH_BF16) {
    if (dm.d == 128) DASH_LAUNCH_AB(__nv_bfloat16, 128); else DASH_LAUNCH_AB(__nv_bfloat16, 64);
  } else {
    if (dm.d == 128) DASH_LAUNCH_AB(float, 128); else DASH_LAUNCH_AB(float, 64);
  }
#undef DASH_LAUNCH_AB
  count_launch();
  return cudaGetLastError();
}

}  // namespace dash
