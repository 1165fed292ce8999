// Shared declarations of the DashAttention CUDA library (internal; the public ABI is include/dash_attn.h).
#pragma once

#include <atomic>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dash_attn.h"

namespace dash {

// Derived problem description handed to kernels by value.
struct Dims {
  int batch, seq_q, seq_kv, h_q, h_kv, d, B, g_q;
  int dtype;    // dash_dtype of Q, K, V, O
  int T_s;      // complete chunks (those with summaries): seq_kv / B
  int T_a;      // all chunks: ceil(seq_kv / B)
  int W;        // mask words per row: ceil(T_a / 32)
  int decode;   // 1: one query row per sequence at kv_len[b]-1
  int causal;        // 1: the paper's setting; 0: every row sees every complete chunk (prefill only)
  int local_blocks;  // window chunks before the own chunk: attended with bias 0, not scored
  int e_int;    // 1/(alpha-1) when it is 1, 2 or 4 (alpha = 2, 1.5, 1.25); 0 otherwise
  float e;      // 1/(alpha-1)
  float x_scale;   // gamma (alpha-1) / sqrt(d): chunk logit scale (Algorithm 2, step 1)
  float sm_scale;  // 1 / sqrt(d): token logit scale (Eq. 1)
  float inv_sigma;
  long long qs[3], ks[3], vs[3], os[3];
  long long list_rows;  // list entries per (batch, KV head)
  // Paged KV cache (decode only): K / V are pools [num_pages, page_size, h_kv, d] (ks / vs = strides of page, token,
  // head) and logical page lp of sequence b is physical page page_table[b * max_pages + lp].  nullptr: contiguous.
  const int* page_table;
  int page_size, max_pages, num_pages;
};

// Where KV token t of sequence b lives: address = first * stride[0] + tok * stride[1] (+ head * stride[2]).  A chunk
// and a 64-token sub-block never straddle a page (page_size is a multiple of both).
__device__ inline void kv_locate(const Dims& dm, int b, int t, int* first, int* tok) {
  if (dm.page_table) {
    const int lp = t / dm.page_size;
    *first = __ldg(dm.page_table + (long long)b * dm.max_pages + lp);
    *tok = t - lp * dm.page_size;
  } else {
    *first = b;
    *tok = t;
  }
}

// Start of row i's list region inside its (batch, KV head) slab.
__host__ __device__ inline long long list_row_offset(const Dims& dm, int i) {
  if (dm.decode) return 0;
  if (!dm.causal) return (long long)i * dm.T_s;
  long long c = i / dm.B;
  return (long long)dm.B * c * (c - 1) / 2 + (long long)(i % dm.B) * c;
}

// Workspace: 256-byte header (status word first), then regions carved by the host.
struct StatusBlock {
  int status;        // dash_status written by kernels (first error wins)
  int detail;        // where it happened (kernel-specific code)
  unsigned int tile_counter;  // persistent-kernel work queue
  int pad[61];
};
static_assert(sizeof(StatusBlock) == 256, "status block is the first 256 bytes of the workspace");
// Behind the status block the workspace holds arrival counters, one per (batch, KV head), for kernels whose last
// thread block of a group finishes the group's work (split-KV decode: the last split merges).  They are zero
// between launches: the block that sees the last arrival clears its counter, and resetting the status word
// clears them all.  Groups beyond the capacity fall back to a separate merge kernel.
constexpr int ARRIVAL_COUNTERS = 4096;
constexpr size_t STATUS_REGION_BYTES = 256 + ARRIVAL_COUNTERS * sizeof(int);
__host__ __device__ inline int* arrival_counters(StatusBlock* sb) { return reinterpret_cast<int*>(sb + 1); }

__device__ inline void report_error(StatusBlock* sb, int status, int detail) {
  if (!sb) return;
  if (atomicCAS(&sb->status, 0, status) == 0) sb->detail = detail;
}

// Bounds checks of everything a kernel indexes with values it read from device memory (list entries, counts): compiled
// in with -DDASH_DEBUG (the debug library), absent from the production build, which trusts the routing outputs it is
// handed.  A failed check records DASH_ERR_CAPACITY with a site code in the status word (when the call has one) and
// runs `fallback`, which must avoid the access; it never traps.
#ifdef DASH_DEBUG
// no do-while wrapper: `fallback` may be a `continue` or `break` of the loop the check sits in
#define DASH_CHECK(cond, sb, code, fallback)     \
  if (!(cond)) {                                 \
    report_error(sb, DASH_ERR_CAPACITY, code);   \
    fallback;                                    \
  } else                                         \
    ((void)0)
#else
#define DASH_CHECK(cond, sb, code, fallback) ((void)0)
#endif

template <typename T> __device__ inline float to_f32(T v);
template <> __device__ inline float to_f32<float>(float v) { return v; }
template <> __device__ inline float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ inline T from_f32(float v);
template <> __device__ inline float from_f32<float>(float v) { return v; }
template <> __device__ inline __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Load 4 consecutive elements as float4 (pointer 8-byte aligned for bf16, 16 for fp32).
__device__ inline float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ inline float4 load4(const __nv_bfloat16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}
__device__ inline void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ inline void store4(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<unsigned int*>(&a);
  u.y = *reinterpret_cast<unsigned int*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// m^e for the integer exponents of alpha = 2, 1.5, 1.25; powf otherwise.  m >= 0.
__device__ __forceinline__ float pow_e(float m, int e_int, float e) {
  if (e_int == 1) return m;
  if (e_int == 2) return m * m;
  if (e_int == 4) { float s = m * m; return s * s; }
  return m > 0.f ? __powf(m, e) : 0.f;
}
// m^(e-1)
__device__ __forceinline__ float pow_em1(float m, int e_int, float e) {
  if (e_int == 1) return m > 0.f ? 1.f : 0.f;
  if (e_int == 2) return m;
  if (e_int == 4) return m * m * m;
  return m > 0.f ? __powf(m, e - 1.f) : 0.f;
}

// Newton on f(tau) = sum [x - tau]_+^e - 1 stops once f <= this: the sum itself carries about 1e-6 of fp32
// rounding noise, and f'(tau) <= -1 at the root for every alpha > 1 (sum m^e = 1 implies sum m^(e-1) >= 1), so the
// threshold is then within 4e-6 of the root; iterating on noise only burns passes.
constexpr float NEWTON_F_TOL = 4e-6f;

// Newton step for the threshold, taken on h(tau) = F(tau)^(1/e) - 1 with F = sum [x - tau]_+^e (G = sum [x - tau]_+^(e-1)):
// tau += (F - F^(1-1/e)) / G.  h has the root of F - 1 and is convex and decreasing like it (it is the e-norm of the
// positive parts, minus one), so the iterates still rise monotonically from the left and one step from the right
// lands on the left; but h is close to linear far from the root, where a step on F - 1 only gains a factor
// 1 - 1/e of the distance, so the same tolerance is reached in about half the passes.  Near the root the two steps
// agree to first order ((F - 1) / (e G)).
__device__ __forceinline__ float newton_delta(float F, float G, int e_int, float e) {
  if (e_int == 1) return (F - 1.f) / G;
  if (e < 1.f) return (F - 1.f) / (e * G);              // alpha > 2: h is no norm, keep the step on F - 1
  if (e_int == 2) return (F - sqrtf(F)) / G;
  if (e_int == 4) return (F - F * rsqrtf(sqrtf(F))) / G;    // F^(3/4)
  return (F - __powf(F, 1.f - 1.f / e)) / G;
}

// ---- chained launches (programmatic dependent launch).  The kernels of one forward pass run back to back on one
// stream, each consuming what the previous one wrote.  Launched through launch_chained, a kernel's thread blocks
// may become resident while the previous kernel drains; chain_wait() then holds them until that kernel has
// completed and its writes are visible, so it must come before the first global access (reads of the previous
// kernel's output and writes to anything it may still read alike).  chain_release() lets the NEXT kernel's blocks
// start arriving once every block of this grid has called it.  Without the launch attribute both are no-ops.
#ifdef __CUDACC__
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// cudaFuncSetAttribute applies to the current device only, and a process may drive several GPUs: one bit per
// device remembers where a kernel's dynamic shared-memory limit has already been raised.
template <typename Kern>
inline cudaError_t allow_dynamic_smem(Kern kern, size_t bytes, std::atomic<unsigned long long>& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && ((done.load(std::memory_order_relaxed) >> dev) & 1ull)) return cudaSuccess;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && tracked) done.fetch_or(1ull << dev, std::memory_order_relaxed);
  return e;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif

void count_launch();
// Host-side switches for the tests (set through dash_attn_test_hooks; the defaults are what production runs with).
struct TestHooks {
  long long wait_limit_cycles = 2000000000LL;   // how long a bounded device-side wait may spin (about 1 s)
  int skip_own_k_load = 0;                      // 1: the prefill attention kernel never loads its first K tile
};
TestHooks& test_hooks();
// Host-side checks shared by the entry points that live outside api.cu.
int validate_params(const dash_params* p, Dims* dm);
int validate_device();

// Launchers (one per translation unit).  All return a cudaError_t from the launch.
// planes non-null: also writes the three bf16 planes (hi + mid + lo = fp32 value) the tensor-core routing kernel
// reads, [3][batch * h_kv * T_s][d], so that no separate split pass is needed
cudaError_t launch_summaries(const Dims& dm, const void* K, const float* qbar, long long qbar_chunk_stride,
                             const int* kv_len, int first_block, int num_blocks, float* Kbar, void* planes,
                             cudaStream_t st);
size_t select_smem_bytes(const Dims& dm, int* tq_out);
// planes_ready: `scratch` already holds the bf16 planes of Kbar (written by launch_summaries)
cudaError_t launch_select(const Dims& dm, const void* Q, const float* Kbar, const int* kv_len, uint32_t* mask,
                          int* count, int* blk_idx, float* blk_bias, float* tau, void* scratch, float* xscratch,
                          StatusBlock* sb, cudaStream_t st, bool planes_ready = false);
size_t select_decode_scratch_bytes(const Dims& dm);
bool select_decode_supported(const Dims& dm);
cudaError_t launch_select_decode(const Dims& dm, const void* Q, const float* Kbar, const int* kv_len, uint32_t* mask,
                                 int* count, int* blk_idx, float* blk_bias, float* tau, float* scratch,
                                 cudaStream_t st);
int select_sm100_token_limit(const Dims& dm);
size_t select_sm100_scratch_bytes(const Dims& dm);
cudaError_t launch_select_sm100(const Dims& dm, int token_limit, const void* Q, const float* Kbar, void* planes,
                                uint32_t* mask, int* count, int* blk_idx, float* blk_bias, float* tau,
                                StatusBlock* sb, cudaStream_t st, bool planes_ready = false);
cudaError_t launch_attend_prefill_generic(const Dims& dm, const void* Q, const void* K, const void* V,
                                          const uint32_t* mask, const float* blk_bias, void* O, cudaStream_t st);
cudaError_t launch_attend_prefill_bwd_generic(const Dims& dm, const void* Q, const void* K, const void* V,
                                              const void* dO, const uint32_t* mask, const float* blk_bias, void* dQ,
                                              float* dK, float* dV, float* dbias, cudaStream_t st);
cudaError_t launch_route_bwd(const Dims& dm, const void* Q, const float* Kbar, const int* count, const int* blk_idx,
                             const float* tau, const float* dbias, float* dQr, float* dKbar, cudaStream_t st);
cudaError_t launch_summaries_bwd(const Dims& dm, const void* K, const float* qbar, long long qbar_chunk_stride,
                                 const float* dKbar, float* dK, float* dqbar, size_t dqbar_bytes, cudaStream_t st);
int decode_num_splits(const Dims& dm);
size_t decode_partial_bytes(const Dims& dm);
cudaError_t launch_attend_decode(const Dims& dm, const void* Q, const void* K, const void* V, const int* kv_len,
                                 const int* count, const int* blk_idx, const float* blk_bias, void* O,
                                 float* partials, StatusBlock* sb, cudaStream_t st);
cudaError_t launch_attend_decode_ex(const Dims& dm, const void* Q, const void* K, const void* V, const int* kv_len,
                                    const int* count, const int* blk_idx, const float* blk_bias, void* O,
                                    float* partials, StatusBlock* sb, cudaStream_t st);
int decode_sm100_min_splits(const Dims& dm);
// O non-null: the last split of every (batch, KV head) merges the partials itself (needs sb's arrival counters)
cudaError_t launch_decode_sm100(const Dims& dm, int n_split, const void* Q, const void* K, const void* V,
                                const int* kv_len, const int* count, const int* blk_idx, const float* blk_bias,
                                float* partials, void* O, StatusBlock* sb, cudaStream_t st);
bool prefill_sm100_supported(const Dims& dm);
// inputs_stable: Q, K, V were not written by the kernel launched just before on the stream
cudaError_t launch_attend_prefill_sm100(const Dims& dm, const void* Q, const void* K, const void* V,
                                        const uint32_t* mask, const float* blk_bias, void* O, StatusBlock* sb,
                                        bool inputs_stable, cudaStream_t st, float* lse2 = nullptr,
                                        float* delta = nullptr, const void* dO = nullptr);
// Stage 2 backward on tensor cores (bf16, head_dim 128, chunks of 64 or 128 tokens, g_q >= 2); scratch: lse2 and delta
// [batch][KV head][query tile][128] floats, prefix [batch * h_kv * seq_q][W] ints.
bool prefill_bwd_sm100_supported(const Dims& dm);
cudaError_t launch_attend_prefill_bwd_sm100(const Dims& dm, const void* Q, const void* K, const void* V, const void* dO,
                                            const uint32_t* mask, const float* blk_bias, float* lse2, float* delta,
                                            int* prefix, void* dQ, float* dK, float* dV, float* dbias, StatusBlock* sb,
                                            cudaStream_t st);

}  // namespace dash
