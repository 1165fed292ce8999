// Stage 0: chunk summaries (Eq. 3, Algorithm 1).
//
// One warp per (batch, KV head, chunk).  A key row (head_dim elements) is read by the whole warp with
// one coalesced vector load per lane; the keys double as values, so the chunk is read from HBM exactly
// once (Algorithm 1 steps 3-6 in one pass).  With a summary query the softmax over the chunk's B keys
// is evaluated online (running max / normaliser); without one the summary is the arithmetic mean.
// HBM-bound: B*d*sizeof(T) bytes read and d*4 bytes written per chunk.
#include "common.cuh"

namespace dash {

constexpr int SUM_WARPS = 8;
constexpr int SUM_UNROLL = 8;

template <typename T, int D>
__global__ void __launch_bounds__(SUM_WARPS * 32)
summaries_kernel(Dims dm, const T* __restrict__ K, const float* __restrict__ qbar, long long qbar_chunk_stride,
                 const int* __restrict__ kv_len, int first_block, int num_blocks, float* __restrict__ Kbar,
                 __nv_bfloat16* __restrict__ planes, long long plane_elems) {
  constexpr int VPL = D / 32;  // elements per lane: 2 (d=64) or 4 (d=128)
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * SUM_WARPS + (threadIdx.x >> 5);
  const long long total = (long long)dm.batch * dm.h_kv * num_blocks;
  chain_wait();       // before any exit: the kernel behind this one relies on it having outlasted its predecessor
  chain_release();
  if (warp >= total) return;
  const int c = first_block + (int)(warp % num_blocks);
  const int r = (int)((warp / num_blocks) % dm.h_kv);
  const int b = (int)(warp / ((long long)num_blocks * dm.h_kv));
  const int len = kv_len ? min(kv_len[b], dm.seq_kv) : dm.seq_kv;
  if ((long long)(c + 1) * dm.B > len) return;  // chunk not complete: no summary (Algorithm 1 step 1)

  int kfirst, ktok;
  kv_locate(dm, b, c * dm.B, &kfirst, &ktok);       // contiguous cache: (b, c * B); paged: (physical page, offset in it)
  const T* kp = K + (long long)kfirst * dm.ks[0] + (long long)ktok * dm.ks[1] + (long long)r * dm.ks[2] + lane * VPL;
  float acc[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) acc[v] = 0.f;

  auto loadv = [&](const T* p, float* out) {
    if constexpr (VPL == 4) {
      float4 f = load4(p);
      out[0] = f.x; out[1] = f.y; out[2] = f.z; out[3] = f.w;
    } else {
      out[0] = to_f32<T>(p[0]); out[1] = to_f32<T>(p[1]);
    }
  };

  if (qbar == nullptr) {
    // plain mean: 16 rows in flight per warp (a small prefill has fewer warps than the SMs can hold, so the depth
    // of each warp's load queue is what covers the DRAM latency)
    constexpr int MU = 2 * SUM_UNROLL;
    for (int t0 = 0; t0 < dm.B; t0 += MU) {
      float kv[MU][VPL];
#pragma unroll
      for (int u = 0; u < MU; ++u) loadv(kp + (long long)min(t0 + u, dm.B - 1) * dm.ks[1], kv[u]);
#pragma unroll
      for (int u = 0; u < MU; ++u)
        if (t0 + u < dm.B) {
#pragma unroll
          for (int v = 0; v < VPL; ++v) acc[v] += kv[u][v];
        }
    }
    const float inv = 1.f / (float)dm.B;
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[v] *= inv;
  } else {
    float q[VPL];
    const float* qp = qbar + (long long)c * qbar_chunk_stride + (long long)r * D + lane * VPL;
#pragma unroll
    for (int v = 0; v < VPL; ++v) q[v] = qp[v] * dm.sm_scale;
    float m = -INFINITY, l = 0.f;
    for (int t0 = 0; t0 < dm.B; t0 += SUM_UNROLL) {
      float kv[SUM_UNROLL][VPL], s[SUM_UNROLL];
#pragma unroll
      for (int u = 0; u < SUM_UNROLL; ++u) loadv(kp + (long long)(t0 + u) * dm.ks[1], kv[u]);
#pragma unroll
      for (int u = 0; u < SUM_UNROLL; ++u) {
        float p = 0.f;
#pragma unroll
        for (int v = 0; v < VPL; ++v) p += q[v] * kv[u][v];
        s[u] = p;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int u = 0; u < SUM_UNROLL; ++u) s[u] += __shfl_xor_sync(0xffffffffu, s[u], o);
      float mt = m;
#pragma unroll
      for (int u = 0; u < SUM_UNROLL; ++u) mt = fmaxf(mt, s[u]);
      const float corr = __expf(m - mt);  // m = -inf on the first tile: exp(-inf) = 0
      l *= corr;
#pragma unroll
      for (int v = 0; v < VPL; ++v) acc[v] *= corr;
#pragma unroll
      for (int u = 0; u < SUM_UNROLL; ++u) {
        const float p = __expf(s[u] - mt);
        l += p;
#pragma unroll
        for (int v = 0; v < VPL; ++v) acc[v] += p * kv[u][v];
      }
      m = mt;
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[v] *= inv;
  }
  const long long at = (((long long)b * dm.h_kv + r) * dm.T_s + c) * D + lane * VPL;
  float* op = Kbar + at;
#pragma unroll
  for (int v = 0; v < VPL; ++v) op[v] = acc[v];
  if (planes) {
    // x = hi + mid + lo exactly (three bf16 roundings of the successive remainders)
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      const float x = acc[v];
      const __nv_bfloat16 hi = __float2bfloat16_rn(x);
      const float r1 = x - __bfloat162float(hi);
      const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
      const float r2 = r1 - __bfloat162float(mid);
      planes[at + v] = hi;
      planes[plane_elems + at + v] = mid;
      planes[2 * plane_elems + at + v] = __float2bfloat16_rn(r2);
    }
  }
}

cudaError_t launch_summaries(const Dims& dm, const void* K, const float* qbar, long long qbar_chunk_stride,
                             const int* kv_len, int first_block, int num_blocks, float* Kbar, void* planes,
                             cudaStream_t st) {
  if (num_blocks <= 0) return cudaSuccess;
  const long long plane_elems = (long long)dm.batch * dm.h_kv * dm.T_s * dm.d;
  const long long total = (long long)dm.batch * dm.h_kv * num_blocks;
  const unsigned grid = (unsigned)((total + SUM_WARPS - 1) / SUM_WARPS);
  const dim3 block(SUM_WARPS * 32);
  cudaError_t le = cudaSuccess;
#define DASH_LAUNCH_SUM(T, D)                                                                               \
  le = launch_chained(summaries_kernel<T, D>, dim3(grid), block, 0, st, dm, (const T*)K, qbar,              \
                      qbar_chunk_stride, kv_len, first_block, num_blocks, Kbar, (__nv_bfloat16*)planes, plane_elems)
  if (dm.B % SUM_UNROLL != 0) return cudaErrorInvalidValue;
  if (dm.dtype == DASH_BF16) {
    if (dm.d == 128) DASH_LAUNCH_SUM(__nv_bfloat16, 128); else DASH_LAUNCH_SUM(__nv_bfloat16, 64);
  } else {
    if (dm.d == 128) DASH_LAUNCH_SUM(float, 128); else DASH_LAUNCH_SUM(float, 64);
  }
  count_launch();
  return le;
#undef DASH_LAUNCH_SUM
}

}  // namespace dash
