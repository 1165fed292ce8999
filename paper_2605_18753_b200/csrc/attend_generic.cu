// Stage 2, prefill, CUDA-core path (Eq. 7 in the form of Proposition 1; Algorithm 3).
//
// Used for fp32 tensors and for shapes the tensor-core kernel does not cover.  One warp per
// (batch, query token, query head): it walks the set bits of the row's mask words in ascending chunk
// order, takes the next entry of the row's bias list for every routed chunk (0 for the own chunk, which
// also gets the causal mask, Algorithm 3 step 7) and runs the online softmax of Algorithm 3 steps 8-11.
// Lanes own keys for the logits and head_dim slices for the output accumulator.
#include "common.cuh"

namespace dash {

constexpr int AG_WARPS = 4;

template <typename T, int D>
__global__ void __launch_bounds__(AG_WARPS * 32)
attend_prefill_generic_kernel(Dims dm, const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                              const uint32_t* __restrict__ mask, const float* __restrict__ blk_bias,
                              T* __restrict__ O) {
  constexpr int VPL = D / 32;
  __shared__ __align__(16) float qs[AG_WARPS][D];
  __shared__ float ps[AG_WARPS][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long gw = (long long)blockIdx.x * AG_WARPS + warp;
  const long long total = (long long)dm.batch * dm.seq_q * dm.h_q;
  chain_wait();
  chain_release();
  if (gw >= total) return;
  const int h = (int)(gw % dm.h_q);
  const int i = dm.seq_q - 1 - (int)((gw / dm.h_q) % dm.seq_q);  // long rows first
  const int b = (int)(gw / ((long long)dm.h_q * dm.seq_q));
  const int r = h / dm.g_q;
  const int c_own = dm.causal ? i / dm.B : dm.T_s;   // non-causal: the incomplete tail chunk, seen whole by every row

  const T* qp = Q + (long long)b * dm.qs[0] + (long long)i * dm.qs[1] + (long long)h * dm.qs[2];
  for (int k = lane; k < D; k += 32) qs[warp][k] = to_f32<T>(qp[k]) * dm.sm_scale;
  __syncwarp();

  const T* kbase = K + (long long)b * dm.ks[0] + (long long)r * dm.ks[2];
  const T* vbase = V + (long long)b * dm.vs[0] + (long long)r * dm.vs[2];
  const uint32_t* mrow = mask + (((long long)b * dm.h_kv + r) * dm.seq_q + i) * dm.W;
  const float* brow = blk_bias + ((long long)b * dm.h_kv + r) * dm.list_rows + list_row_offset(dm, i);

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
      if (c > c_own) continue;  // a mask that marks a future chunk is ignored (causal)
      const float bias = (c == c_own) ? 0.f : brow[cursor];
      if (c != c_own) ++cursor;
      const int t_end = (c == c_own && dm.causal) ? (i + 1) : min((c + 1) * dm.B, dm.seq_kv);
      for (int t0 = c * dm.B; t0 < t_end; t0 += 32) {
        const int t = t0 + lane;
        float s = -INFINITY;
        if (t < t_end) {
          const T* kp = kbase + (long long)t * dm.ks[1];
          float a = 0.f;
#pragma unroll 4
          for (int k = 0; k < D; k += 4) {
            const float4 kv = load4(kp + k);
            const float4 qv = *reinterpret_cast<const float4*>(&qs[warp][k]);
            a = fmaf(qv.x, kv.x, a); a = fmaf(qv.y, kv.y, a); a = fmaf(qv.z, kv.z, a); a = fmaf(qv.w, kv.w, a);
          }
          s = a + bias;
        }
        const float mt = fmaxf(m, warp_max(s));
        const float corr = __expf(m - mt);
        const float p = (t < t_end) ? __expf(s - mt) : 0.f;
        l = l * corr + warp_sum(p);
#pragma unroll
        for (int v = 0; v < VPL; ++v) acc[v] *= corr;
        ps[warp][lane] = p;
        __syncwarp();
        const int nt = min(32, t_end - t0);
        for (int u = 0; u < nt; ++u) {
          const float pu = ps[warp][u];
          const T* vp = vbase + (long long)(t0 + u) * dm.vs[1] + lane * VPL;
          if constexpr (VPL == 4) {
            const float4 vv = load4(vp);
            acc[0] = fmaf(pu, vv.x, acc[0]); acc[1] = fmaf(pu, vv.y, acc[1]);
            acc[2] = fmaf(pu, vv.z, acc[2]); acc[3] = fmaf(pu, vv.w, acc[3]);
          } else {
            acc[0] = fmaf(pu, to_f32<T>(vp[0]), acc[0]);
            acc[1] = fmaf(pu, to_f32<T>(vp[1]), acc[1]);
          }
        }
        __syncwarp();
        m = mt;
      }
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  T* op = O + (long long)b * dm.os[0] + (long long)i * dm.os[1] + (long long)h * dm.os[2] + lane * VPL;
#pragma unroll
  for (int v = 0; v < VPL; ++v) op[v] = from_f32<T>(acc[v] * inv);
}

cudaError_t launch_attend_prefill_generic(const Dims& dm, const void* Q, const void* K, const void* V,
                                          const uint32_t* mask, const float* blk_bias, void* O, cudaStream_t st) {
  const long long total = (long long)dm.batch * dm.seq_q * dm.h_q;
  const unsigned grid = (unsigned)((total + AG_WARPS - 1) / AG_WARPS);
  cudaError_t le = cudaSuccess;
#define DASH_LAUNCH_AG(T, D)                                                                                    \
  le = launch_chained(attend_prefill_generic_kernel<T, D>, dim3(grid), dim3(AG_WARPS * 32), 0, st, dm,          \
                      (const T*)Q, (const T*)K, (const T*)V, mask, blk_bias, (T*)O)
  if (dm.dtype == DASH_BF16) {
    if (dm.d == 128) DASH_LAUNCH_AG(__nv_bfloat16, 128); else DASH_LAUNCH_AG(__nv_bfloat16, 64);
  } else {
    if (dm.d == 128) DASH_LAUNCH_AG(float, 128); else DASH_LAUNCH_AG(float, 64);
  }
#undef DASH_LAUNCH_AG
  count_launch();
  return le;
}

}  // namespace dash
