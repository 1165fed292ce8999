// Stage 1: alpha-entmax chunk routing (Eq. 2, Eq. 4, Algorithm 2, Proposition 1).
//
// One thread block handles TQ consecutive query tokens of one (batch, KV head); the TQ*g_q (token, head)
// rows share their candidate chunks because a tile never straddles a chunk boundary.
//   1. Chunk logits x = gamma(alpha-1) <q, kbar_c>/sqrt(d) for every row and candidate chunk are computed
//      in fp32 and kept in shared memory (they are never written to HBM, unlike Algorithm 2 step 1).
//   2. One warp per token: for each head of the group, the threshold tau is found by Newton's method on
//      f(tau) = sum [x - tau]_+^e - 1 (e = 1/(alpha-1)), started at max(x) - 1 where f >= 0.  f is convex
//      and decreasing, so the iterates rise monotonically to the root and never pass it; for alpha = 2
//      the iteration is finite.  For alpha in {2, 1.5, 1.25} the powers are products (no exp/log).
//   3. Group weights w_c = mean_h [x_hc - tau_h]_+^e, support bit = (max_h (x_hc - tau_h) > 0), 32 chunks
//      per ballot = one mask word (Algorithm 2 steps 7-13); log w in a scaled form; mu = mean log w;
//      bias = (log w - mu)/sigma compacted into the row's list (steps 15-19), the own chunk's bit is set.
// With a local window of L chunks the last L chunks before the own one are not scored: their bits are set and
// they close the row's list with bias 0 (they take no part in tau, w or mu).
#include "common.cuh"

namespace dash {

constexpr int SEL_THREADS = 256;
constexpr int SEL_CT = 64;          // candidate chunks per staged tile of summaries
constexpr int SEL_SMEM_BUDGET = 200 * 1024;
constexpr int SEL_MAX_NEWTON = 64;
constexpr int SEL_MAX_NEWTON_GENERIC = 400;

struct SelectPlan {
  int TQ;         // tokens per block
  int r_pad;      // rows of the score tile (4, 8, 16, 32)
  int xs_stride;  // floats per score row in shared memory
  size_t smem;
};

static bool plan_select(const Dims& dm, SelectPlan* pl) {
  if (dm.g_q > 32) return false;
  int tq = 1;
  if (!dm.decode) {
    while (tq * 2 * dm.g_q <= 32 && tq * 2 <= dm.B) tq *= 2;
  }
  const int max_cand = (dm.decode || !dm.causal) ? dm.T_s : min(dm.T_s, (dm.seq_q - 1) / dm.B);
  const int xs = ((max_cand + SEL_CT - 1) / SEL_CT) * SEL_CT + 4;
  for (;; tq /= 2) {
    const int rows = tq * dm.g_q;
    const int r_pad = rows <= 4 ? 4 : rows <= 8 ? 8 : rows <= 16 ? 16 : 32;
    const size_t smem = ((size_t)r_pad * xs + (size_t)r_pad * (dm.d + 4) + (size_t)SEL_CT * (dm.d + 4) + 64) * 4;
    if (smem <= (size_t)SEL_SMEM_BUDGET) {
      pl->TQ = tq; pl->r_pad = r_pad; pl->xs_stride = xs; pl->smem = smem;
      return true;
    }
    if (tq == 1) return false;
  }
}

size_t select_smem_bytes(const Dims& dm, int* tq_out) {
  SelectPlan pl;
  if (!plan_select(dm, &pl)) return 0;
  if (tq_out) *tq_out = pl.TQ;
  return pl.smem;
}

// RPT rows x CPT chunks per thread; CX = 64/CPT threads along chunks, RY = 256/CX along rows.
template <typename T, int D, int RPT, int CPT>
__global__ void __launch_bounds__(SEL_THREADS)
select_kernel(Dims dm, int TQ, int xs_stride, int token_base, const T* __restrict__ Q, const float* __restrict__ Kbar,
              const int* __restrict__ kv_len, uint32_t* __restrict__ mask, int* __restrict__ count,
              int* __restrict__ blk_idx, float* __restrict__ blk_bias, float* __restrict__ tau_out) {
  constexpr int CX = SEL_CT / CPT;
  constexpr int RY = SEL_THREADS / CX;
  constexpr int R_PAD = RY * RPT;
  constexpr int DS = D + 4;  // padded row stride (floats) of the staged Q and summary tiles
  extern __shared__ __align__(16) float smem[];
  float* Xs = smem;                                  // [R_PAD][xs_stride]
  float* Qs = Xs + (size_t)R_PAD * xs_stride;        // [R_PAD][DS]
  float* Ks = Qs + R_PAD * DS;                       // [SEL_CT][DS]
  float* taus = Ks + SEL_CT * DS;                    // [R_PAD]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile = gridDim.x - 1 - blockIdx.x;       // late (long) rows first
  const int r = blockIdx.y, b = blockIdx.z;
  const int g_q = dm.g_q;
  const int rows = TQ * g_q;
  chain_wait();
  chain_release();

  int i0, c_own;
  if (dm.decode) {
    int L = kv_len ? kv_len[b] : dm.seq_kv;
    L = max(1, min(L, dm.seq_kv));
    i0 = 0;
    c_own = (L - 1) / dm.B;
  } else {
    i0 = token_base + tile * TQ;
    // non-causal: every complete chunk is a candidate of every row; the incomplete tail chunk (index T_s, if
    // the length is not a multiple of the chunk size) plays the own chunk's part: attended with bias 0
    c_own = dm.causal ? i0 / dm.B : dm.T_s;
  }
  const bool has_own = c_own < dm.T_a;
  const int n_vis = min(c_own, dm.T_s);                 // chunks before the own one: routed candidates, then the window
  const int n_cand = max(n_vis - dm.local_blocks, 0);   // scored by entmax

  // ---- stage the query rows in fp32 (row = token * g_q + head-in-group)
  for (int idx = tid; idx < R_PAD * (D / 4); idx += SEL_THREADS) {
    const int row = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row < rows) {
      const int t = row / g_q, hh = row % g_q;
      const int i = i0 + t;
      if (dm.decode || i < dm.seq_q) {
        const T* qp = Q + (long long)b * dm.qs[0] + (dm.decode ? 0 : (long long)i * dm.qs[1]) +
                      (long long)(r * g_q + hh) * dm.qs[2] + c4;
        v = load4(qp);
      }
    }
    store4(Qs + row * DS + c4, v);
  }

  // ---- chunk logits, SEL_CT candidates at a time
  const int tx = tid % CX, ty = tid / CX;
  const float* kb = Kbar + ((long long)b * dm.h_kv + r) * dm.T_s * D;
  for (int c0 = 0; c0 < n_cand; c0 += SEL_CT) {
    __syncthreads();  // previous tile consumed (and Qs visible on the first pass)
    for (int idx = tid; idx < SEL_CT * (D / 4); idx += SEL_THREADS) {
      const int cr = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (c0 + cr < n_cand) v = load4(kb + (long long)(c0 + cr) * D + c4);
      store4(Ks + cr * DS + c4, v);
    }
    __syncthreads();
    float acc[RPT][CPT];
#pragma unroll
    for (int k = 0; k < RPT; ++k)
#pragma unroll
      for (int j = 0; j < CPT; ++j) acc[k][j] = 0.f;
#pragma unroll 4
    for (int dd = 0; dd < D; dd += 4) {
      float4 qv[RPT], kv[CPT];
#pragma unroll
      for (int k = 0; k < RPT; ++k) qv[k] = load4(Qs + (ty * RPT + k) * DS + dd);
#pragma unroll
      for (int j = 0; j < CPT; ++j) kv[j] = load4(Ks + (tx + j * CX) * DS + dd);
#pragma unroll
      for (int k = 0; k < RPT; ++k)
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
          acc[k][j] = fmaf(qv[k].x, kv[j].x, acc[k][j]);
          acc[k][j] = fmaf(qv[k].y, kv[j].y, acc[k][j]);
          acc[k][j] = fmaf(qv[k].z, kv[j].z, acc[k][j]);
          acc[k][j] = fmaf(qv[k].w, kv[j].w, acc[k][j]);
        }
    }
#pragma unroll
    for (int k = 0; k < RPT; ++k)
#pragma unroll
      for (int j = 0; j < CPT; ++j)
        Xs[(size_t)(ty * RPT + k) * xs_stride + c0 + tx + j * CX] = acc[k][j] * dm.x_scale;
  }
  __syncthreads();

  // ---- one warp per token: thresholds, group weights, mask words, bias list
  const int e_int = dm.e_int;
  const float e = dm.e;
  const int max_it = e_int ? SEL_MAX_NEWTON : SEL_MAX_NEWTON_GENERIC;
  const float log_gq = logf((float)g_q);
  for (int t = warp; t < TQ; t += SEL_THREADS / 32) {
    const int i = i0 + t;
    if (!dm.decode && i >= dm.seq_q) continue;
    const long long row_id = ((long long)b * dm.h_kv + r) * dm.seq_q + (dm.decode ? 0 : i);
    float* x0 = Xs + (size_t)(t * g_q) * xs_stride;

    for (int hh = 0; hh < g_q; ++hh) {
      const float* x = x0 + (size_t)hh * xs_stride;
      float tau = 0.f;
      if (n_cand > 0) {
        float mx = -INFINITY;
        for (int c = lane; c < n_cand; c += 32) mx = fmaxf(mx, x[c]);
        mx = warp_max(mx);
        tau = mx - 1.f;
        for (int it = 0; it < max_it; ++it) {
          float f = 0.f, g = 0.f;
          for (int c = lane; c < n_cand; c += 32) {
            const float m = x[c] - tau;
            if (m > 0.f) {
              f += pow_e(m, e_int, e);
              g += pow_em1(m, e_int, e);
            }
          }
          f = warp_sum(f) - 1.f;
          g = warp_sum(g);
          if (!(f > NEWTON_F_TOL)) break;
          const float nt = tau + newton_delta(f + 1.f, g, e_int, e);
          if (!(nt > tau)) break;
          tau = nt;
        }
      }
      if (lane == 0) {
        taus[t * g_q + hh] = tau;
        if (tau_out) tau_out[((long long)b * dm.h_q + r * g_q + hh) * dm.seq_q + (dm.decode ? 0 : i)] = tau;
      }
    }
    __syncwarp();

    // pass 1: support, log w (stashed over head 0's logits), mask words
    uint32_t* mrow = mask + row_id * dm.W;
    float slog = 0.f;
    int nsel = 0;
    uint32_t myword = 0;
    for (int j = 0; j < dm.W; ++j) {
      const int c = j * 32 + lane;
      bool sel = false;
      float lw = INFINITY;
      if (c < n_cand) {
        float mstar = 0.f;
        for (int hh = 0; hh < g_q; ++hh) mstar = fmaxf(mstar, x0[(size_t)hh * xs_stride + c] - taus[t * g_q + hh]);
        if (mstar > 0.f) {
          sel = true;
          float s = 0.f;
          const float inv = 1.f / mstar;
          for (int hh = 0; hh < g_q; ++hh) {
            const float m = fmaxf(x0[(size_t)hh * xs_stride + c] - taus[t * g_q + hh], 0.f);
            s += pow_e(m * inv, e_int, e);
          }
          lw = e * logf(mstar) + logf(s) - log_gq;
          slog += lw;
        }
        x0[c] = lw;  // +inf marks "not routed"
      }
      uint32_t word = __ballot_sync(0xffffffffu, sel);
      nsel += __popc(word);
      const bool local = c >= n_cand && c < n_vis;
      if (local) x0[c] = -INFINITY;  // -inf marks a window chunk: listed with bias 0
      word |= __ballot_sync(0xffffffffu, local);
      if (has_own && (c_own >> 5) == j) word |= 1u << (c_own & 31);
      if (lane == (j & 31)) myword = word;
      if ((j & 31) == 31 || j == dm.W - 1) {
        if (lane <= (j & 31)) mrow[(j & ~31) + lane] = myword;
      }
    }
    slog = warp_sum(slog);
    if (lane == 0) count[row_id] = nsel + (n_vis - n_cand);

    // pass 2: bias = (log w - mu) / sigma, compacted in ascending chunk order
    if (nsel + (n_vis - n_cand) > 0) {
      const float mu = nsel > 0 ? slog / (float)nsel : 0.f;
      const long long loff = ((long long)b * dm.h_kv + r) * dm.list_rows + list_row_offset(dm, i);
      int base = 0;
      for (int j = 0; j * 32 < n_vis; ++j) {
        const int c = j * 32 + lane;
        const float lw = (c < n_vis) ? x0[c] : INFINITY;
        const bool sel = lw < INFINITY;
        const uint32_t word = __ballot_sync(0xffffffffu, sel);
        if (sel) {
          const long long pos = loff + base + __popc(word & ((1u << lane) - 1u));
          blk_bias[pos] = lw == -INFINITY ? 0.f : (lw - mu) * dm.inv_sigma;
          if (blk_idx) blk_idx[pos] = c;
        }
        base += __popc(word);
      }
    }
  }
}

template <typename T, int D, int RPT, int CPT>
static cudaError_t launch_one(const Dims& dm, const SelectPlan& pl, int token_base, const void* Q, const float* Kbar,
                              const int* kv_len, uint32_t* mask, int* count, int* blk_idx, float* blk_bias,
                              float* tau, cudaStream_t st) {
  auto kern = select_kernel<T, D, RPT, CPT>;
  static std::atomic<unsigned long long> configured{0};
  if (cudaError_t e = allow_dynamic_smem(kern, SEL_SMEM_BUDGET, configured); e != cudaSuccess) return e;
  const int tiles = dm.decode ? 1 : (dm.seq_q - token_base + pl.TQ - 1) / pl.TQ;
  dim3 grid(tiles, dm.h_kv, dm.batch);
  cudaError_t le = launch_chained(kern, grid, dim3(SEL_THREADS), pl.smem, st, dm, pl.TQ, pl.xs_stride, token_base,
                                  (const T*)Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau);
  count_launch();
  return le;
}

template <typename T, int D>
static cudaError_t launch_rows(const Dims& dm, const SelectPlan& pl, int token_base, const void* Q, const float* Kbar,
                               const int* kv_len, uint32_t* mask, int* count, int* blk_idx, float* blk_bias,
                               float* tau, cudaStream_t st) {
  switch (pl.r_pad) {
    case 32: return launch_one<T, D, 2, 4>(dm, pl, token_base, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau, st);
    case 16: return launch_one<T, D, 1, 4>(dm, pl, token_base, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau, st);
    case 8:  return launch_one<T, D, 1, 2>(dm, pl, token_base, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau, st);
    default: return launch_one<T, D, 1, 1>(dm, pl, token_base, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau, st);
  }
}

cudaError_t launch_select(const Dims& dm, const void* Q, const float* Kbar, const int* kv_len, uint32_t* mask,
                          int* count, int* blk_idx, float* blk_bias, float* tau, void* scratch, float* xscratch,
                          StatusBlock* sb, cudaStream_t st, bool planes_ready) {
  // decode: streaming score kernel + per-(batch, KV head) routing kernel
  if (dm.decode && xscratch && select_decode_supported(dm))
    return launch_select_decode(dm, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau, xscratch, st);
  // bf16 prefill rows whose candidates fit in tensor memory go to the tcgen05 kernel; everything else
  // (fp32, decode, very long rows) to the CUDA-core kernel below
  int token_base = 0;
  const int tc_tokens = scratch ? select_sm100_token_limit(dm) : 0;
  if (tc_tokens > 0) {
    cudaError_t e = launch_select_sm100(dm, tc_tokens, Q, Kbar, scratch, mask, count, blk_idx, blk_bias, tau, sb, st,
                                        planes_ready);
    if (e != cudaSuccess || tc_tokens >= dm.seq_q) return e;
    token_base = tc_tokens;
  }
  SelectPlan pl;
  if (!plan_select(dm, &pl)) return cudaErrorInvalidConfiguration;
  if (dm.dtype == DASH_BF16) {
    if (dm.d == 128) return launch_rows<__nv_bfloat16, 128>(dm, pl, token_base, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau, st);
    return launch_rows<__nv_bfloat16, 64>(dm, pl, token_base, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau, st);
  }
  if (dm.d == 128) return launch_rows<float, 128>(dm, pl, token_base, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau, st);
  return launch_rows<float, 64>(dm, pl, token_base, Q, Kbar, kv_len, mask, count, blk_idx, blk_bias, tau, st);
}

}  // namespace dash
