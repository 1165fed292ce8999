// Stage 2 backward, prefill, tensor-core path for sm_100a (Section 3.5: the backward pass reuses the forward pass's bit
// mask; Eq. 7 in the form of Proposition 1 is what is differentiated, with the routing held fixed).
//
// With P = softmax of the row's logits l_j = <q,k_j>/sqrt(d) + bias_c(j) over its selected tokens, dP = dO V^T,
// delta = <O, dO> per row and dS = P o (dP - delta):
//     dQ = dS K / sqrt(d),   dK = dS^T Q / sqrt(d),   dV = P^T dO,   dbias_c = sum of dS over the chunk's tokens.
// Four launches behind the forward kernel run in "statistics" mode (it leaves the log-sum-exp and delta of every row):
//   mask_prefix_kernel      per row, the number of routed chunks in the mask words before each word (so that a row's
//                           list entry for a chunk can be found from one word of its mask);
//   tile_union_kernel       per query tile, the OR of its rows' mask words (which chunks any of its rows attends);
//   attend_bwd_dq_kernel    query-tile stationary, the forward kernel's walk over the union of the tile's routed
//                           chunks: S = Q K^T and dP = dO V^T into tensor memory, dS (bf16) back into tensor memory,
//                           dQ += dS K accumulated in tensor memory; dbias from the row sums of dS;
//   attend_bwd_dkv_kernel   key-slice stationary (64 keys of one KV head): walks the query tiles that attend the slice
//                           (the tiles of its own chunk, causally masked, then every later tile whose mask holds the
//                           chunk), recomputes S and dP, and accumulates dV^T += dO^T P and dK^T += Q^T dS in tensor
//                           memory (P and dS pass through shared memory as bf16 MN-major operands), so dK and dV need
//                           no atomics and no zeroing.
// bf16 operands, fp32 accumulation; head_dim 128; chunks of 64 or 128 tokens; g_q >= 2.  Every wait is bounded.
#include <cuda.h>

#include <type_traits>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace dash {

namespace {

constexpr int NKV = 64;                 // keys per step / per slice
constexpr int HD = 128;
constexpr uint32_t Q_BYTES = 128 * HD * 2;          // 32 KiB: a 128-row tile, two 128x64 regions
constexpr uint32_t KV_TILE_BYTES = NKV * HD * 2;    // 16 KiB
constexpr int MAX_TQ = 64;
constexpr float LOG2E = 1.4426950408889634f;

struct BwdArgs {
  Dims dm;
  int TQ;             // tokens per query tile
  int n_tiles;        // query tiles per (batch, KV head)
  int n_slices;       // 64-key slices per (batch, KV head)
  long long wait_limit;
  const uint32_t* mask;
  const float* blk_bias;
  const float* lse2;
  const float* delta;
  const int* prefix;
  const uint32_t* tile_union;   // [batch * h_kv][query tile][W]: OR of the tile's rows' mask words
  __nv_bfloat16* dQ;
  float* dK;
  float* dV;
  float* dbias;
  StatusBlock* sb;
};

// prefix[row][w] = routed chunks of the row in mask words 0 .. w-1 (the own chunk's bit, which sits behind every routed
// one, is left out)
__global__ void __launch_bounds__(256)
mask_prefix_kernel(Dims dm, const uint32_t* __restrict__ mask, int* __restrict__ prefix) {
  chain_wait();
  chain_release();
  const long long row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long rows = (long long)dm.batch * dm.h_kv * dm.seq_q;
  if (row >= rows) return;
  const int i = (int)(row % dm.seq_q);
  const int c_own = i / dm.B;
  int acc = 0;
  for (int w = 0; w < dm.W; ++w) {
    prefix[row * dm.W + w] = acc;
    uint32_t word = mask[row * dm.W + w];
    if (w == (c_own >> 5)) word &= (1u << (c_own & 31)) - 1u;
    else if (w > (c_own >> 5)) word = 0u;
    acc += __popc(word);
  }
}

// tile_union[group][tile][w] = OR over the tile's rows of mask word w: which chunks any row of the tile attends
__global__ void __launch_bounds__(256)
tile_union_kernel(Dims dm, int TQ, int n_tiles, const uint32_t* __restrict__ mask, uint32_t* __restrict__ tile_union) {
  chain_wait();
  chain_release();
  const long long warp_id = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const long long total = (long long)dm.batch * dm.h_kv * n_tiles;
  if (warp_id >= total) return;
  const long long grp = warp_id / n_tiles;
  const int tile = (int)(warp_id % n_tiles);
  for (int w = 0; w < dm.W; ++w) {
    uint32_t u = 0u;
    for (int t = lane; t < TQ; t += 32) {
      const int i = tile * TQ + t;
      if (i < dm.seq_q) u |= mask[(grp * dm.seq_q + i) * dm.W + w];
    }
    u = __reduce_or_sync(0xffffffffu, u);
    if (lane == 0) tile_union[warp_id * dm.W + w] = u;
  }
}

// ===================================================================================================================
// dQ and dbias: query-tile stationary
// ===================================================================================================================
namespace dq {

// Two warpgroups form dS, each for half of a step's 64 columns (no row maximum is needed: the log-sum-exp is known), so
// a step's exponentials take half as long.  One issuing thread per product (S, dP, dQ): a thread issues an MMA every
// 60-80 clocks whatever its size, and 20 per step through one thread would be the kernel's pace.
constexpr int W_KPROD = 8, W_S = 9, W_VPROD = 10, W_DP = 11, W_DQ = 12;
constexpr int THREADS = 512;              // 8 dS warps, 5 service warps, 3 idle: whole warpgroups, so that the registers can be re-divided
constexpr int REGS_SERVICE = 56, REGS_SOFTMAX = 200;   // per thread after the re-division (128 each at launch)
static_assert(THREADS == 512 && 256 * (REGS_SOFTMAX - 128) <= 256 * (128 - REGS_SERVICE),
              "the dS warpgroups can only take what the service warpgroups released: a larger request never completes");
constexpr int KST = 3;                  // K / V ring and S / dP ring: stage = step mod 3, held until the step's dQ product is done
constexpr uint32_t TMEM_COLS = 512;     // S [0,192) dP [192,384) dQ [384,512)
constexpr uint32_t COL_DP = 192, COL_DQ = 384;
enum Bar { QD_FULL = 0, META, S_FULL = 2, DP_FULL = 5, DS_FULL = 8, V_FULL = 11, K_FULL = 14, KV_FREE = 17, N_BARS = 20 };
struct Misc {
  unsigned long long bar[N_BARS];
  uint32_t tmem_base;
  int n_steps;
  int abort_flag;
  int kvbase[KST];
  float bias[KST][MAX_TQ];
  long long entry[KST][MAX_TQ];         // list entry of the token for the step's chunk (-1: none: own chunk or not routed)
};
constexpr uint32_t OFF_Q = 0, OFF_DO = OFF_Q + Q_BYTES, OFF_K = OFF_DO + Q_BYTES, OFF_V = OFF_K + KST * KV_TILE_BYTES,
                   OFF_MISC = OFF_V + KST * KV_TILE_BYTES, SMEM = OFF_MISC + sizeof(Misc);
static_assert(SMEM <= 232448, "one block per SM");

__global__ void __launch_bounds__(THREADS, 1)
attend_bwd_dq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmDO,
                     const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, BwdArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  Misc* misc = reinterpret_cast<Misc*>(smem + OFF_MISC);
  const Dims& dm = a.dm;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t sbase = ptx::smem_u32(smem);
  auto bar = [&](int i) { return ptx::smem_u32(&misc->bar[i]); };
  volatile int* abort_flag = &misc->abort_flag;
  const long long wait_limit = a.wait_limit;
  auto wait_on = [&](uint32_t barrier, uint32_t parity) { return ptx::mbar_wait(barrier, parity, abort_flag, wait_limit); };

  const int groups = dm.batch * dm.h_kv;
  const int tile = a.n_tiles - 1 - (int)(blockIdx.x / groups);  // late (long) tiles first
  const int grp = (int)(blockIdx.x % groups);
  const int b = grp / dm.h_kv, r = grp % dm.h_kv;
  const int TQ = a.TQ, g_q = dm.g_q;
  const int i0 = tile * TQ;
  const int c_own = i0 / dm.B;
  const int sub_per_blk = dm.B / NKV;
  const int own_steps = (i0 % dm.B) / NKV + 1;

  if (tid == 0) {
    misc->abort_flag = ((sbase & 1023u) != 0u) ? 1 : 0;
    if (misc->abort_flag) report_error(a.sb, DASH_ERR_CUDA, 110);
    ptx::mbar_init(bar(QD_FULL), 1);
    ptx::mbar_init(bar(META), 1);
    for (int s = 0; s < KST; ++s) {
      ptx::mbar_init(bar(S_FULL + s), 1);
      ptx::mbar_init(bar(DP_FULL + s), 1);
      ptx::mbar_init(bar(DS_FULL + s), 256);
      ptx::mbar_init(bar(K_FULL + s), 1);
      ptx::mbar_init(bar(V_FULL + s), 1);
      ptx::mbar_init(bar(KV_FREE + s), 1);
    }
    ptx::fence_barrier_init();
  }
  if (warp == W_S) {
    ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), TMEM_COLS);
    ptx::tmem_relinquish();
    ptx::tc_fence_before();
  }
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = misc->tmem_base;
  chain_wait();
  chain_release();
  if (a.sb && *reinterpret_cast<volatile int*>(&a.sb->status) != 0) *abort_flag = 1;
  __syncthreads();

  auto load_kv = [&](const CUtensorMap* tm, uint32_t dst, uint32_t barrier, int kv0) {
    ptx::mbar_arrive_expect_tx(barrier, KV_TILE_BYTES);
    ptx::tma_load_4d(dst, tm, barrier, 0, r, kv0, b);
    ptx::tma_load_4d(dst + KV_TILE_BYTES / 2, tm, barrier, 64, r, kv0, b);
  };

  if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE));
  if (warp == W_KPROD || warp == W_VPROD) {
    // =========================== producers: the forward kernel's walk ===========================
    const bool do_k = (warp == W_KPROD), do_v = (warp == W_VPROD);
    if (lane == 0 && do_k) {
      ptx::prefetch_tensormap(&tmQ);
      ptx::prefetch_tensormap(&tmDO);
      ptx::prefetch_tensormap(&tmK);
      ptx::prefetch_tensormap(&tmV);
      ptx::mbar_arrive_expect_tx(bar(QD_FULL), 2 * Q_BYTES);
      ptx::tma_load_4d(sbase + OFF_Q, &tmQ, bar(QD_FULL), 0, r * g_q, i0, b);
      ptx::tma_load_4d(sbase + OFF_Q + Q_BYTES / 2, &tmQ, bar(QD_FULL), 64, r * g_q, i0, b);
      ptx::tma_load_4d(sbase + OFF_DO, &tmDO, bar(QD_FULL), 0, r * g_q, i0, b);
      ptx::tma_load_4d(sbase + OFF_DO + Q_BYTES / 2, &tmDO, bar(QD_FULL), 64, r * g_q, i0, b);
    }
    // own chunk first (steps 0 .. own_steps-1 <= 2 go to stages 0 / 1, which are free)
    for (int sub = 0; sub < own_steps; ++sub) {
      const int kv0 = c_own * dm.B + sub * NKV;
      if (do_k) {
        if (lane == 0) load_kv(&tmK, sbase + OFF_K + sub * KV_TILE_BYTES, bar(K_FULL + sub), kv0);
      } else {
        for (int t = lane; t < TQ; t += 32) { misc->bias[sub][t] = 0.f; misc->entry[sub][t] = -1; }
        if (lane == 0) misc->kvbase[sub] = kv0;
        __syncwarp();
        if (lane == 0) load_kv(&tmV, sbase + OFF_V + sub * KV_TILE_BYTES, bar(V_FULL + sub), kv0);
      }
    }
    const int n_words = (c_own >> 5) + 1;
    const long long row0 = ((long long)b * dm.h_kv + r) * dm.seq_q;
    const uint32_t own_word_keep = (c_own & 31) == 31 ? 0xffffffffu : ((2u << (c_own & 31)) - 1u);
    auto load_rows = [&](int w, uint32_t* rw) {
      for (int q = 0; q < 2; ++q) {
        const int t = lane + 32 * q;
        rw[q] = (t < TQ && i0 + t < dm.seq_q) ? a.mask[(row0 + i0 + t) * dm.W + w] : 0u;
      }
    };
    auto union_of = [&](int w, const uint32_t* rw) -> uint32_t {
      uint32_t u = __reduce_or_sync(0xffffffffu, rw[0] | rw[1]);
      if (w == n_words - 1) u = (u & own_word_keep) | (1u << (c_own & 31));
      return u;
    };
    int total = 0;
    for (int w = 0; w < n_words; ++w) {
      uint32_t rw[2];
      load_rows(w, rw);
      total += __popc(union_of(w, rw));
    }
    const int n_steps = (total - 1) * sub_per_blk + own_steps;
    if (lane == 0 && do_k) {
      misc->n_steps = n_steps;
      ptx::mbar_arrive(bar(META));
    }
    long long loff[2];
    for (int q = 0; q < 2; ++q) {
      const int t = lane + 32 * q;
      const int i = min(i0 + t, dm.seq_q - 1);
      loff[q] = ((long long)b * dm.h_kv + r) * dm.list_rows + list_row_offset(dm, i);
    }
    int j = own_steps;
    bool ok = true;
    int last_j[KST];
    for (int s = 0; s < KST; ++s) last_j[s] = s < own_steps ? s : -1;
    int seen[2] = {0, 0};
    uint32_t rw[2], rw_n[2] = {0u, 0u};
    load_rows(0, rw);
    if (n_words > 1) load_rows(1, rw_n);
    for (int w = 0; w < n_words && ok; ++w) {
      uint32_t u = union_of(w, rw);
      uint32_t rb[2];
      for (int q = 0; q < 2; ++q) rb[q] = w == n_words - 1 ? rw[q] & own_word_keep & ~(1u << (c_own & 31)) : rw[q];
      while (u != 0u && ok) {
        const int bit = __ffs(u) - 1;
        u &= u - 1;
        const int c = w * 32 + bit;
        if (c == c_own) break;                   // last of the walk, done first
        float bv[2];
        long long en[2];
        for (int q = 0; q < 2; ++q) {
          const bool member = do_v && ((rb[q] >> bit) & 1u);
          const long long e = loff[q] + seen[q] + __popc(rb[q] & ((1u << bit) - 1u));
          bv[q] = member ? __ldg(a.blk_bias + e) : -INFINITY;
          en[q] = member ? e : -1;
        }
        for (int sub = 0; sub < sub_per_blk && ok; ++sub, ++j) {
          const int kv0 = c * dm.B + sub * NKV;
          const int st = j % KST;
          if (j >= KST) ok = wait_on(bar(KV_FREE + st), (uint32_t)(j / KST - 1) & 1u);   // every product of step j-3 has read the stage
          if (!ok) break;
          if (do_k) {
            if (lane == 0) load_kv(&tmK, sbase + OFF_K + st * KV_TILE_BYTES, bar(K_FULL + st), kv0);
          } else {
            for (int q = 0; q < 2; ++q) {
              const int t = lane + 32 * q;
              if (t < TQ) { misc->bias[st][t] = bv[q]; misc->entry[st][t] = en[q]; }
            }
            if (lane == 0) misc->kvbase[st] = kv0;
            __syncwarp();
            if (lane == 0) load_kv(&tmV, sbase + OFF_V + st * KV_TILE_BYTES, bar(V_FULL + st), kv0);
          }
          last_j[st] = j;
        }
      }
      seen[0] += __popc(rb[0]);
      seen[1] += __popc(rb[1]);
      rw[0] = rw_n[0]; rw[1] = rw_n[1];
      if (w + 2 < n_words) load_rows(w + 2, rw_n);
    }
    if (!ok && lane == 0) {
      for (int s = 0; s < KST; ++s) {
        if (last_j[s] < 0) continue;
        const uint32_t full = bar((do_k ? K_FULL : V_FULL) + s), parity = (uint32_t)(last_j[s] / KST) & 1u;
        for (int k = 0; k < 200000 && !ptx::mbar_try_wait(full, parity); ++k) {}
      }
      if (do_k)
        for (int k = 0; k < 200000 && !ptx::mbar_try_wait(bar(QD_FULL), 0); ++k) {}
    }
  } else if (warp == W_S || warp == W_DP) {
    // =========================== issuers of S = Q K^T (warp W_S) and dP = dO V^T (warp W_DP) ===========================
    // Ring slot j mod 3 of S / dP is free when the K / V stage of the same index is: both wait for the dQ product of
    // step j-3 (the producers do, before they refill the stage).
    if (lane == 0) {
      const bool is_s = warp == W_S;
      bool ok = wait_on(bar(QD_FULL), 0);
      int n_steps = 0x7fffffff;            // known from step 1 on; step 0 (the own chunk) always exists
      constexpr uint32_t IDESC_S = ptx::idesc_bf16_f32(128, NKV, false, false);
      const uint64_t ad0 = ptx::smem_desc_sw128(sbase + (is_s ? OFF_Q : OFF_DO), 16, 1024);
      const uint64_t bd0 = ptx::smem_desc_sw128(sbase + (is_s ? OFF_K : OFF_V), 16, 1024);
      const uint32_t col0 = is_s ? 0u : COL_DP;
      for (int j = 0; j < n_steps && ok; ++j) {
        if (j == 1) {
          ok = wait_on(bar(META), 0);
          if (!ok) break;
          n_steps = misc->n_steps;
          if (j >= n_steps) break;
        }
        const int st = j % KST;
        ok = wait_on(bar((is_s ? K_FULL : V_FULL) + st), (uint32_t)(j / KST) & 1u);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint64_t bd = bd0 + (uint64_t)((st * KV_TILE_BYTES) >> 4);
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          const uint64_t off_a = (uint64_t)(((k >> 2) * (Q_BYTES / 2) + (k & 3) * 32) >> 4);
          const uint64_t off_b = (uint64_t)(((k >> 2) * (KV_TILE_BYTES / 2) + (k & 3) * 32) >> 4);
          ptx::mma_bf16_ss(tmem + col0 + st * NKV, ad0 + off_a, bd + off_b, IDESC_S, k > 0 ? 1u : 0u);
        }
        ptx::mma_commit(bar((is_s ? S_FULL : DP_FULL) + st));
      }
    }
    __syncwarp();
  } else if (warp == W_DQ) {
    // =========================== issuer of dQ += dS K ===========================
    if (lane == 0) {
      bool ok = true;
      int n_steps = 0x7fffffff;
      constexpr uint32_t IDESC_DQ = ptx::idesc_bf16_f32(128, HD, false, true);
      const uint64_t kmn0 = ptx::smem_desc_sw128(sbase + OFF_K, KV_TILE_BYTES / 2, 1024);   // K as MN-major B
      for (int j = 0; j < n_steps && ok; ++j) {
        if (j == 1) {
          ok = wait_on(bar(META), 0);
          if (!ok) break;
          n_steps = misc->n_steps;
          if (j >= n_steps) break;
        }
        const int st = j % KST;
        ok = wait_on(bar(DS_FULL + st), (uint32_t)(j / KST) & 1u);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint64_t kmn = kmn0 + (uint64_t)((st * KV_TILE_BYTES) >> 4);
#pragma unroll
        for (int k = 0; k < NKV / 16; ++k)
          // dS of keys 16k .. 16k+15: eight packed columns, keys 0-31 at columns 0-15 and keys 32-63 at columns 32-47
          ptx::mma_bf16_ts(tmem + COL_DQ, tmem + st * NKV + (k >> 1) * 32 + (k & 1) * 8, kmn + (uint64_t)((k * 16 * 128) >> 4),
                           IDESC_DQ, (j > 0 || k > 0) ? 1u : 0u);
        ptx::mma_commit(bar(KV_FREE + st));
      }
    }
    __syncwarp();
  }
  } else {
    // =========================== dS / epilogue: thread = tile row, warpgroup = column half ===========================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX));
    const int wg = warp >> 2;
    const int m = (warp & 3) * 32 + lane;
    const int t = m / g_q, hh = m % g_q;
    const int i_row = i0 + t;
    const bool row_ok = i_row < dm.seq_q;
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const float c1 = dm.sm_scale * LOG2E;
    const long long srow = (((long long)b * dm.h_kv + r) * a.n_tiles + tile) * 128 + m;
    const float lse2 = row_ok ? a.lse2[srow] : 0.f;
    const float delta = row_ok ? a.delta[srow] : 0.f;
    bool ok = true;
    int n_steps = 0x7fffffff;              // known from step 1 on; step 0 (the own chunk) always exists
    for (int j = 0; j < n_steps && ok; ++j) {
      if (j == 1) {
        ok = wait_on(bar(META), 0);
        if (!ok) break;
        n_steps = misc->n_steps;
        if (j >= n_steps) break;
      }
      const int st = j % KST;
      const uint32_t ph = (uint32_t)(j / KST) & 1u;
      ok = wait_on(bar(V_FULL + st), ph);                  // bias / entry / kvbase of the step visible
      if (!ok) break;
      const float bias = row_ok ? misc->bias[st][t] : -INFINITY;
      const long long entry = misc->entry[st][t];
      const int kv0 = misc->kvbase[st];
      ok = wait_on(bar(S_FULL + st), ph) && wait_on(bar(DP_FULL + st), ph);
      if (!ok) break;
      ptx::tc_fence_after();
      const int n_vis = i_row - kv0 + 1;                   // causal: column c visible iff c < n_vis
      const float off = bias * LOG2E - lse2;               // -inf: the row did not route the chunk
      float rowsum = 0.f;
      {
        const int half = wg;
        uint32_t sv[32], gv[32];
        DASH_TMEM_LD32(sv, lane_addr + st * NKV + half * 32);
        DASH_TMEM_LD32(gv, lane_addr + COL_DP + st * NKV + half * 32);
        ptx::tmem_wait_ld();
        uint32_t packed[16];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          float ds[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const bool vis = half * 32 + c + u < n_vis;
            const float p = vis ? exp2f(fmaf(__uint_as_float(sv[c + u]), c1, off)) : 0.f;
            ds[u] = p * (__uint_as_float(gv[c + u]) - delta);
            rowsum += ds[u];
          }
          __nv_bfloat162 h = __floats2bfloat162_rn(ds[0], ds[1]);
          packed[c >> 1] = *reinterpret_cast<uint32_t*>(&h);
        }
        // dS row -> the first 16 columns of this warpgroup's own half of the step's S buffer (two bf16 per column):
        // the other warpgroup's scores, in the other 32 columns, are never touched
        ptx::tmem_st_n<16>(lane_addr + st * NKV + half * 32, packed);
      }
      ptx::tmem_wait_st();
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar(DS_FULL + st));
      // dbias of the (token, chunk): the row sums of the group's heads (adjacent lanes) added up
      for (int o = 1; o < g_q; o <<= 1) rowsum += __shfl_xor_sync(0xffffffffu, rowsum, o);
      if (hh == 0 && entry >= 0 && row_ok) atomicAdd(a.dbias + entry, rowsum);
    }
    // epilogue: dQ / sqrt(d) -> global; each warpgroup takes half of the row's columns
    if (ok && n_steps > 0) ok = wait_on(bar(KV_FREE + ((n_steps - 1) % KST)), (uint32_t)((n_steps - 1) / KST) & 1u);
    if (ok && n_steps > 0) {
      ptx::tc_fence_after();
      __nv_bfloat16* op = a.dQ + (long long)b * dm.qs[0] + (long long)i_row * dm.qs[1] + (long long)(r * g_q + hh) * dm.qs[2];
      const float sc = dm.sm_scale;
#pragma unroll 1
      for (int q = wg * 2; q < wg * 2 + 2; ++q) {
        uint32_t o[32];
        DASH_TMEM_LD32(o, lane_addr + COL_DQ + q * 32);
        ptx::tmem_wait_ld();
        if (row_ok) {
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            uint4 v;
            __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(o[c]) * sc, __uint_as_float(o[c + 1]) * sc);
            __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(o[c + 2]) * sc, __uint_as_float(o[c + 3]) * sc);
            __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(o[c + 4]) * sc, __uint_as_float(o[c + 5]) * sc);
            __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(o[c + 6]) * sc, __uint_as_float(o[c + 7]) * sc);
            v.x = *reinterpret_cast<uint32_t*>(&h0); v.y = *reinterpret_cast<uint32_t*>(&h1);
            v.z = *reinterpret_cast<uint32_t*>(&h2); v.w = *reinterpret_cast<uint32_t*>(&h3);
            *reinterpret_cast<uint4*>(op + q * 32 + c) = v;
          }
        }
      }
    }
    ptx::tc_fence_before();
  }

  __syncthreads();
  if (warp == W_S) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, TMEM_COLS);
  }
  if (tid == 0 && misc->abort_flag) report_error(a.sb, DASH_ERR_TIMEOUT, 111);
}

}  // namespace dq

// ===================================================================================================================
// dK and dV: key-slice stationary
// ===================================================================================================================
namespace dkv {

// Two warpgroups form P and dS, each for half of the slice's keys on every step (no row maximum is needed, so the halves
// are independent and a step's P / dS stretch takes half as long); one issuing thread per product: 32 MMAs per step
// are too many for one.  W_PROD loads the tiles, W_META looks up the per-token biases of each step; W_SD issues S,
// W_DP dP, W_ACC dV^T, W_DK dK^T.
constexpr int W_PROD = 8, W_SD = 9, W_ACC = 10, W_DP = 11, W_DK = 12, W_META = 13;
constexpr int THREADS = 512;              // 8 P / dS warps, 6 service warps, 2 idle: whole warpgroups
constexpr int REGS_SERVICE = 80, REGS_SOFTMAX = 176;     // (the bias and loader warps need more than the issuers)
static_assert(THREADS == 512 && 256 * (REGS_SOFTMAX - 128) <= 256 * (128 - REGS_SERVICE), "see the dQ kernel");
constexpr uint32_t TMEM_COLS = 512;     // S0 S1 [0,128) dP0 dP1 [128,256) dV^T [256,320) dK^T [320,384)
constexpr uint32_t COL_DP = 128, COL_DV = 256, COL_DK = 320;
constexpr uint32_t PS_BYTES = 128 * NKV * 2;       // 16 KiB: P (or dS) of a step, 128 rows of 128 bytes
enum Bar { KV_FULL = 0, QD_FULL = 1, SD_FULL = 3, ACC_DONE = 5, PDS_FULL = 7, N_BARS = 9 };   // SD_FULL, ACC_DONE: two arrivals (one per issuer)
struct Misc {
  unsigned long long bar[N_BARS];
  uint32_t tmem_base;
  int abort_flag;
  int total;                            // number of steps, written with the end marker
  int tile[2];                          // query tile of the stage's step (-1: no more steps)
  float bias[2][MAX_TQ];                // per token of the tile: the chunk's bias (-inf: the token does not attend it)
  alignas(16) float lse2[2][128];       // the tile's row statistics (bulk copies)
  alignas(16) float delta[2][128];
};
constexpr uint32_t OFF_K = 0, OFF_V = OFF_K + KV_TILE_BYTES, OFF_Q = OFF_V + KV_TILE_BYTES,   // Q stage s at OFF_Q + s * 2 * Q_BYTES,
                   OFF_P = OFF_Q + 4 * Q_BYTES, OFF_DS = OFF_P + PS_BYTES,                   //   its dO tile Q_BYTES behind
                   OFF_MISC = OFF_DS + PS_BYTES, SMEM = OFF_MISC + sizeof(Misc);
static_assert(SMEM <= 232448, "one block per SM");

__global__ void __launch_bounds__(THREADS, 1)
attend_bwd_dkv_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmDO,
                      const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, BwdArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  Misc* misc = reinterpret_cast<Misc*>(smem + OFF_MISC);
  const Dims& dm = a.dm;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t sbase = ptx::smem_u32(smem);
  auto bar = [&](int i) { return ptx::smem_u32(&misc->bar[i]); };
  volatile int* abort_flag = &misc->abort_flag;
  const long long wait_limit = a.wait_limit;
  auto wait_on = [&](uint32_t barrier, uint32_t parity) { return ptx::mbar_wait(barrier, parity, abort_flag, wait_limit); };

  const int groups = dm.batch * dm.h_kv;
  const int slice = (int)(blockIdx.x / groups);                  // early slices first: every later token may attend them
  const int grp = (int)(blockIdx.x % groups);
  const int b = grp / dm.h_kv, r = grp % dm.h_kv;
  const int TQ = a.TQ, g_q = dm.g_q;
  const int k0 = slice * NKV;                                    // first key of the slice
  const int c = k0 / dm.B;                                       // its chunk

  if (tid == 0) {
    misc->abort_flag = ((sbase & 1023u) != 0u) ? 1 : 0;
    if (misc->abort_flag) report_error(a.sb, DASH_ERR_CUDA, 120);
    ptx::mbar_init(bar(KV_FULL), 1);
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(bar(QD_FULL + s), 2);     // the loader's arrival (with the byte count) and the bias warp's
      ptx::mbar_init(bar(SD_FULL + s), 2);
      ptx::mbar_init(bar(ACC_DONE + s), 2);
      ptx::mbar_init(bar(PDS_FULL + s), 256);
    }
    ptx::fence_barrier_init();
  }
  if (warp == W_SD) {
    ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), TMEM_COLS);
    ptx::tmem_relinquish();
    ptx::tc_fence_before();
  }
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = misc->tmem_base;
  chain_wait();
  chain_release();
  if (a.sb && *reinterpret_cast<volatile int*>(&a.sb->status) != 0) *abort_flag = 1;
  __syncthreads();

  if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE));
  if (warp == W_PROD || warp == W_META) {
    // =========================== producers ===========================
    // Both warps enumerate the slice's steps in the same order: (i) the tiles of the slice's own chunk that can see it
    // (tokens from k0 on: bias 0, causal mask in the kernel), (ii) the later tiles one of whose rows routed the chunk,
    // read 32 tiles at a time from the tile unions.  W_PROD fetches K / V once and the Q / dO tiles and row
    // statistics of every step; W_META looks up the per-token biases.  A step's stage is free once both accumulating
    // products of step j-2 have completed.
    const bool loader = warp == W_PROD;
    if (lane == 0 && loader) {
      ptx::prefetch_tensormap(&tmQ);
      ptx::prefetch_tensormap(&tmDO);
      ptx::prefetch_tensormap(&tmK);
      ptx::prefetch_tensormap(&tmV);
      ptx::mbar_arrive_expect_tx(bar(KV_FULL), 2 * KV_TILE_BYTES);
      ptx::tma_load_4d(sbase + OFF_K, &tmK, bar(KV_FULL), 0, r, k0, b);
      ptx::tma_load_4d(sbase + OFF_K + KV_TILE_BYTES / 2, &tmK, bar(KV_FULL), 64, r, k0, b);
      ptx::tma_load_4d(sbase + OFF_V, &tmV, bar(KV_FULL), 0, r, k0, b);
      ptx::tma_load_4d(sbase + OFF_V + KV_TILE_BYTES / 2, &tmV, bar(KV_FULL), 64, r, k0, b);
    }
    const long long grp_l = (long long)b * dm.h_kv + r;
    const long long row0 = grp_l * dm.seq_q;
    const long long list0 = grp_l * dm.list_rows;
    const long long stat0 = grp_l * a.n_tiles * 128;
    const uint32_t* tu = a.tile_union + grp_l * a.n_tiles * dm.W;
    const int wc = c >> 5, bit = c & 31;
    int j = 0;
    bool ok = true;
    auto stage_free = [&]() {
      if (j >= 2) ok = wait_on(bar(ACC_DONE + (j & 1)), (uint32_t)((j >> 1) - 1) & 1u);
      return ok;
    };
    // ---- the loader's step
    auto load_step = [&](int tile_idx) {
      if (!stage_free()) return;
      const int st = j & 1;
      if (lane == 0) {
        misc->tile[st] = tile_idx;
        if (tile_idx >= 0) {
          const int i0 = tile_idx * TQ;
          const uint32_t dst = sbase + OFF_Q + st * 2 * Q_BYTES;
          ptx::mbar_arrive_expect_tx(bar(QD_FULL + st), 2 * Q_BYTES + 2 * 512);
          ptx::tma_load_4d(dst, &tmQ, bar(QD_FULL + st), 0, r * g_q, i0, b);
          ptx::tma_load_4d(dst + Q_BYTES / 2, &tmQ, bar(QD_FULL + st), 64, r * g_q, i0, b);
          ptx::tma_load_4d(dst + Q_BYTES, &tmDO, bar(QD_FULL + st), 0, r * g_q, i0, b);
          ptx::tma_load_4d(dst + Q_BYTES + Q_BYTES / 2, &tmDO, bar(QD_FULL + st), 64, r * g_q, i0, b);
          ptx::bulk_load(ptx::smem_u32(&misc->lse2[st][0]), a.lse2 + stat0 + (long long)tile_idx * 128, 512, bar(QD_FULL + st));
          ptx::bulk_load(ptx::smem_u32(&misc->delta[st][0]), a.delta + stat0 + (long long)tile_idx * 128, 512, bar(QD_FULL + st));
        } else {
          ptx::mbar_arrive(bar(QD_FULL + st));
        }
      }
      ++j;
    };
    // ---- the bias warp's steps, four at a time: the mask words and prefix counts of all four, then their biases,
    // then the four hand-overs (lane t owns tokens t and t + 32 of a tile)
    int pend[4], n_pend = 0;
    bool pend_own = false;
    auto flush = [&]() {
      float bv[4][2];
      if (pend_own) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
          for (int q = 0; q < 2; ++q) bv[u][q] = (u < n_pend && pend[u] * TQ + lane + 32 * q < dm.seq_q) ? 0.f : -INFINITY;
      } else {
        uint32_t wd[4][2];
        int pf[4][2];
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int t = lane + 32 * q, i = (u < n_pend ? pend[u] : 0) * TQ + t;
            const bool live = u < n_pend && t < TQ && i < dm.seq_q;
            wd[u][q] = live ? a.mask[(row0 + i) * dm.W + wc] : 0u;
            pf[u][q] = live ? a.prefix[(row0 + i) * dm.W + wc] : 0;
          }
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            bv[u][q] = -INFINITY;
            if ((wd[u][q] >> bit) & 1u) {
              const int i = pend[u] * TQ + lane + 32 * q;
              bv[u][q] = __ldg(a.blk_bias + list0 + list_row_offset(dm, i) + pf[u][q] + __popc(wd[u][q] & ((1u << bit) - 1u)));
            }
          }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (u < n_pend && stage_free()) {
          const int st = j & 1;
          for (int q = 0; q < 2; ++q) {
            const int t = lane + 32 * q;
            if (t < TQ) misc->bias[st][t] = bv[u][q];
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar(QD_FULL + st));
          ++j;
        }
      }
      n_pend = 0;
    };
    auto meta_step = [&](int tile_idx, bool own) {
      if (n_pend > 0 && own != pend_own) flush();
      pend_own = own;
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (u == n_pend) pend[u] = tile_idx;
      if (++n_pend == 4) flush();
    };
    auto step = [&](int tile_idx, bool own) {
      if (loader) load_step(tile_idx); else meta_step(tile_idx, own);
    };
    const int t_own_lo = k0 / TQ, t_first_routed = min(((c + 1) * dm.B + TQ - 1) / TQ, a.n_tiles);
    for (int tl = t_own_lo; tl < t_first_routed && ok; ++tl) step(tl, true);
    auto union_word = [&](int tl0) -> uint32_t {
      const int tl = tl0 + lane;
      return tl < a.n_tiles ? __ldg(tu + (long long)tl * dm.W + wc) : 0u;
    };
    uint32_t uw = t_first_routed < a.n_tiles ? union_word(t_first_routed) : 0u, uw_n = 0u;
    for (int tl0 = t_first_routed; tl0 < a.n_tiles && ok; tl0 += 32) {
      if (tl0 + 32 < a.n_tiles) uw_n = union_word(tl0 + 32);
      uint32_t hits = __ballot_sync(0xffffffffu, ((uw >> bit) & 1u) != 0u);
      while (hits != 0u && ok) {
        const int k = __ffs(hits) - 1;
        hits &= hits - 1;
        step(tl0 + k, false);
      }
      uw = uw_n;
    }
    if (!loader && ok && n_pend > 0) flush();
    // the end marker (every role visits every step, so one is enough): both producers arrive on its stage
    if (ok && loader) {
      if (lane == 0) misc->total = j;
      __syncwarp();
      load_step(-1);
    } else if (ok && stage_free()) {
      if (lane == 0) ptx::mbar_arrive(bar(QD_FULL + (j & 1)));
      ++j;
    }
    if (!ok && lane == 0 && loader) {
      // a wait ran out: let the copies already issued land (bounded) before the block retires
      for (int k = 0; k < 200000 && !ptx::mbar_try_wait(bar(KV_FULL), 0); ++k) {}
      for (int s = 0; s < 2; ++s) {
        const int lj = (j - 1 - s);
        if (lj < 0 || misc->tile[lj & 1] < 0) continue;
        for (int k = 0; k < 200000 && !ptx::mbar_try_wait(bar(QD_FULL + (lj & 1)), (uint32_t)(lj >> 1) & 1u); ++k) {}
      }
    }
  } else if (warp == W_SD || warp == W_DP) {
    // =========================== issuers of the score products: S = Q K^T (W_SD), dP = dO V^T (W_DP) ===========================
    if (lane == 0) {
      const bool is_s = warp == W_SD;
      bool ok = wait_on(bar(KV_FULL), 0);
      constexpr uint32_t IDESC_S = ptx::idesc_bf16_f32(128, NKV, false, false);
      const uint64_t kd0 = ptx::smem_desc_sw128(sbase + OFF_K, 16, 1024);
      const uint64_t vd0 = ptx::smem_desc_sw128(sbase + OFF_V, 16, 1024);
      for (int j = 0; ok; ++j) {
        const int buf = j & 1;
        ok = wait_on(bar(QD_FULL + buf), (uint32_t)(j >> 1) & 1u);
        if (!ok || *reinterpret_cast<volatile int*>(&misc->tile[buf]) < 0) break;
        // the warpgroup of this parity has read S / dP of step j-2
        if (j >= 2) ok = wait_on(bar(PDS_FULL + buf), (uint32_t)((j >> 1) - 1) & 1u);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint64_t qd = ptx::smem_desc_sw128(sbase + OFF_Q + buf * 2 * Q_BYTES, 16, 1024);
        const uint64_t gd = ptx::smem_desc_sw128(sbase + OFF_Q + buf * 2 * Q_BYTES + Q_BYTES, 16, 1024);
        if (is_s) {
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) {
            const uint64_t off_a = (uint64_t)(((k >> 2) * (Q_BYTES / 2) + (k & 3) * 32) >> 4);
            const uint64_t off_b = (uint64_t)(((k >> 2) * (KV_TILE_BYTES / 2) + (k & 3) * 32) >> 4);
            ptx::mma_bf16_ss(tmem + buf * NKV, qd + off_a, kd0 + off_b, IDESC_S, k > 0 ? 1u : 0u);
          }
        } else {
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) {
            const uint64_t off_a = (uint64_t)(((k >> 2) * (Q_BYTES / 2) + (k & 3) * 32) >> 4);
            const uint64_t off_b = (uint64_t)(((k >> 2) * (KV_TILE_BYTES / 2) + (k & 3) * 32) >> 4);
            ptx::mma_bf16_ss(tmem + COL_DP + buf * NKV, gd + off_a, vd0 + off_b, IDESC_S, k > 0 ? 1u : 0u);
          }
        }
        ptx::mma_commit(bar(SD_FULL + buf));
      }
    }
    __syncwarp();
  } else if (warp == W_ACC || warp == W_DK) {
    // =========================== issuers of the accumulating products: dV^T += dO^T P (W_ACC), dK^T += Q^T dS (W_DK) ===========================
    if (lane == 0) {
      const bool is_v = warp == W_ACC;
      constexpr uint32_t IDESC_ACC = ptx::idesc_bf16_f32(128, NKV, true, true);     // A = (Q | dO)^T, B = (dS | P): both MN-major
      const uint64_t pd0 = ptx::smem_desc_sw128(sbase + OFF_P, PS_BYTES, 1024);
      const uint64_t sd0 = ptx::smem_desc_sw128(sbase + OFF_DS, PS_BYTES, 1024);
      bool ok = true;
      for (int j = 0; ok; ++j) {
        const int buf = j & 1;
        ok = wait_on(bar(QD_FULL + buf), (uint32_t)(j >> 1) & 1u);
        if (!ok || *reinterpret_cast<volatile int*>(&misc->tile[buf]) < 0) break;
        ok = wait_on(bar(PDS_FULL + buf), (uint32_t)(j >> 1) & 1u);
        if (!ok) break;
        ptx::tc_fence_after();
        // (Q | dO) tile [row][d] read as MN-major A: M = d (two blocks of 64, Q_BYTES / 2 apart), K = rows (16 rows = 2048 B)
        const uint64_t qmn = ptx::smem_desc_sw128(sbase + OFF_Q + buf * 2 * Q_BYTES, Q_BYTES / 2, 1024);
        const uint64_t gmn = ptx::smem_desc_sw128(sbase + OFF_Q + buf * 2 * Q_BYTES + Q_BYTES, Q_BYTES / 2, 1024);
        if (is_v) {
#pragma unroll
          for (int k = 0; k < 128 / 16; ++k) {
            const uint64_t adv = (uint64_t)((k * 16 * 128) >> 4);
            ptx::mma_bf16_ss(tmem + COL_DV, gmn + adv, pd0 + adv, IDESC_ACC, (j > 0 || k > 0) ? 1u : 0u);
          }
        } else {
#pragma unroll
          for (int k = 0; k < 128 / 16; ++k) {
            const uint64_t adv = (uint64_t)((k * 16 * 128) >> 4);
            ptx::mma_bf16_ss(tmem + COL_DK, qmn + adv, sd0 + adv, IDESC_ACC, (j > 0 || k > 0) ? 1u : 0u);
          }
        }
        ptx::mma_commit(bar(ACC_DONE + buf));
      }
    }
    __syncwarp();
  }
  } else {
    // =========================== P, dS: thread = tile row, warpgroup = half of the keys; epilogue: thread = d ===========================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX));
    const int wg = warp >> 2;
    const int m = (warp & 3) * 32 + lane;
    const int t = m / g_q;
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const float c1 = dm.sm_scale * LOG2E;
    bool ok = true;
    for (int j = 0; ok; ++j) {
      const int buf = j & 1;
      const uint32_t ph = (uint32_t)(j >> 1) & 1u;
      ok = wait_on(bar(QD_FULL + buf), ph);
      if (!ok) break;
      const int tile_idx = *reinterpret_cast<volatile int*>(&misc->tile[buf]);
      if (tile_idx < 0) break;
      const int i_row = tile_idx * TQ + t;
      const bool row_ok = i_row < dm.seq_q;
      const float lse2 = row_ok ? misc->lse2[buf][m] : 0.f;
      const float delta = row_ok ? misc->delta[buf][m] : 0.f;
      const float bias = row_ok ? misc->bias[buf][t] : -INFINITY;
      const float off = bias * LOG2E - lse2;
      const int n_vis = i_row - k0 + 1 - wg * 32;            // visible columns of this warpgroup's half
      ok = wait_on(bar(SD_FULL + buf), ph);
      if (!ok) break;
      ptx::tc_fence_after();
      uint32_t pp[16], dd[16];                               // the row's 32 P and 32 dS values of this half as bf16 pairs
      {
        uint32_t sv[32], gv[32];
        DASH_TMEM_LD32(sv, lane_addr + buf * NKV + wg * 32);
        DASH_TMEM_LD32(gv, lane_addr + COL_DP + buf * NKV + wg * 32);
        ptx::tmem_wait_ld();
#pragma unroll
        for (int cc = 0; cc < 32; cc += 2) {
          float p[2], ds[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const bool vis = cc + u < n_vis;
            p[u] = vis ? exp2f(fmaf(__uint_as_float(sv[cc + u]), c1, off)) : 0.f;
            ds[u] = p[u] * (__uint_as_float(gv[cc + u]) - delta);
          }
          __nv_bfloat162 hp = __floats2bfloat162_rn(p[0], p[1]);
          __nv_bfloat162 hd = __floats2bfloat162_rn(ds[0], ds[1]);
          pp[cc >> 1] = *reinterpret_cast<uint32_t*>(&hp);
          dd[cc >> 1] = *reinterpret_cast<uint32_t*>(&hd);
        }
      }
      // the accumulating products of the step before have read P / dS
      if (j >= 1) ok = wait_on(bar(ACC_DONE + (buf ^ 1)), (uint32_t)((j - 1) >> 1) & 1u);
      if (!ok) break;
      // row m of the [128 rows][64 keys] tiles: 128 bytes, 16-byte pieces swizzled with the row (128-byte swizzle); this
      // warpgroup's keys are pieces 4 wg .. 4 wg + 3
      uint8_t* prow = smem + OFF_P + m * 128;
      uint8_t* drow = smem + OFF_DS + m * 128;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        const int phys = ((wg * 4 + ch) ^ (m & 7)) << 4;
        *reinterpret_cast<uint4*>(prow + phys) = make_uint4(pp[ch * 4], pp[ch * 4 + 1], pp[ch * 4 + 2], pp[ch * 4 + 3]);
        *reinterpret_cast<uint4*>(drow + phys) = make_uint4(dd[ch * 4], dd[ch * 4 + 1], dd[ch * 4 + 2], dd[ch * 4 + 3]);
      }
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar(PDS_FULL + buf));
    }
    // epilogue: dV^T, dK^T [d = TMEM lane][key = column] -> dV, dK [batch][key][KV head][d]; one warpgroup each
    const int n_done = ok ? *reinterpret_cast<volatile int*>(&misc->total) : 0;
    if (ok && n_done > 0) ok = wait_on(bar(ACC_DONE + ((n_done - 1) & 1)), (uint32_t)((n_done - 1) >> 1) & 1u);
    if (ok) {
      ptx::tc_fence_after();
      const int d = m;
      float* out = wg == 0 ? a.dV : a.dK;
      const float mul = wg == 0 ? 1.f : dm.sm_scale;
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
        uint32_t v[32];
        if (n_done > 0) {
          DASH_TMEM_LD32(v, lane_addr + (wg == 0 ? COL_DV : COL_DK) + half * 32);
          ptx::tmem_wait_ld();
        } else {
#pragma unroll
          for (int cc = 0; cc < 32; ++cc) v[cc] = 0u;
        }
#pragma unroll
        for (int cc = 0; cc < 32; ++cc) {
          const int key = k0 + half * 32 + cc;
          if (key < dm.seq_kv)
            out[(((long long)b * dm.seq_kv + key) * dm.h_kv + r) * HD + d] = __uint_as_float(v[cc]) * mul;
        }
      }
    }
    ptx::tc_fence_before();
  }

  __syncthreads();
  if (warp == W_SD) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, TMEM_COLS);
  }
  if (tid == 0 && misc->abort_flag) report_error(a.sb, DASH_ERR_TIMEOUT, 121);
}

}  // namespace dkv

// [batch, tokens, heads, 128] bf16 tensor with element strides s[3]; box = 64 x box_heads x box_tokens x 1.
bool make_map(CUtensorMap* out, const void* base, long long tokens, int heads, int batch, const long long* s,
              int box_heads, int box_tokens) {
  cuuint64_t dims[4] = {(cuuint64_t)HD, (cuuint64_t)heads, (cuuint64_t)tokens, (cuuint64_t)batch};
  auto st = [](long long e) { return (cuuint64_t)((e > 0 ? e : 8) * 2); };
  cuuint64_t strides[3] = {st(s[2]), st(s[1]), st(s[0])};
  cuuint32_t box[4] = {64u, (cuuint32_t)box_heads, (cuuint32_t)box_tokens, 1u};
  return encode_bf16_sw128_4d(out, base, dims, strides, box);
}

}  // namespace

bool prefill_bwd_sm100_supported(const Dims& dm) {
  if (!prefill_sm100_supported(dm)) return false;
  if (dm.d != 128 || (dm.B != 64 && dm.B != 128)) return false;
  if (dm.qs[2] % 8 != 0 || dm.qs[1] % 8 != 0) return false;     // 16-byte stores of dQ rows
  return true;
}

cudaError_t launch_attend_prefill_bwd_sm100(const Dims& dm, const void* Q, const void* K, const void* V, const void* dO,
                                            const uint32_t* mask, const float* blk_bias, float* lse2, float* delta,
                                            int* prefix, void* dQ, float* dK, float* dV, float* dbias, StatusBlock* sb,
                                            cudaStream_t st) {
  // 1. forward recomputation in statistics mode: log-sum-exp and delta of every row (O itself is not written)
  cudaError_t e = launch_attend_prefill_sm100(dm, Q, K, V, mask, blk_bias, nullptr, sb, false, st, lse2, delta, dO);
  if (e != cudaSuccess) return e;
  // 2. routed-chunk counts before every mask word
  const long long rows = (long long)dm.batch * dm.h_kv * dm.seq_q;
  e = launch_chained(mask_prefix_kernel, dim3((unsigned)((rows + 255) / 256)), dim3(256), 0, st, dm, mask, prefix);
  count_launch();
  if (e != cudaSuccess) return e;

  BwdArgs a;
  a.dm = dm;
  a.TQ = 128 / dm.g_q;
  a.n_tiles = (dm.seq_q + a.TQ - 1) / a.TQ;
  a.n_slices = (dm.seq_kv + NKV - 1) / NKV;
  a.wait_limit = test_hooks().wait_limit_cycles;
  a.mask = mask; a.blk_bias = blk_bias; a.lse2 = lse2; a.delta = delta; a.prefix = prefix;
  // the tile unions sit behind the prefix counts in the same scratch region
  uint32_t* tile_union = reinterpret_cast<uint32_t*>(prefix + rows * dm.W);
  a.tile_union = tile_union;
  {
    const long long warps = (long long)dm.batch * dm.h_kv * a.n_tiles;
    e = launch_chained(tile_union_kernel, dim3((unsigned)((warps * 32 + 255) / 256)), dim3(256), 0, st, dm, a.TQ, a.n_tiles,
                       mask, tile_union);
    count_launch();
    if (e != cudaSuccess) return e;
  }
  a.dQ = (__nv_bfloat16*)dQ; a.dK = dK; a.dV = dV; a.dbias = dbias; a.sb = sb;
  CUtensorMap tq, tg, tk, tv;
  if (!make_map(&tq, Q, dm.seq_q, dm.h_q, dm.batch, dm.qs, dm.g_q, a.TQ)) return cudaErrorInvalidValue;
  if (!make_map(&tg, dO, dm.seq_q, dm.h_q, dm.batch, dm.os, dm.g_q, a.TQ)) return cudaErrorInvalidValue;
  if (!make_map(&tk, K, dm.seq_kv, dm.h_kv, dm.batch, dm.ks, 1, NKV)) return cudaErrorInvalidValue;
  if (!make_map(&tv, V, dm.seq_kv, dm.h_kv, dm.batch, dm.vs, 1, NKV)) return cudaErrorInvalidValue;
  const int groups = dm.batch * dm.h_kv;
  {
    static std::atomic<unsigned long long> configured{0};
    if ((e = allow_dynamic_smem(dq::attend_bwd_dq_kernel, dq::SMEM, configured)) != cudaSuccess) return e;
    e = launch_chained(dq::attend_bwd_dq_kernel, dim3((unsigned)((long long)a.n_tiles * groups)), dim3(dq::THREADS),
                       dq::SMEM, st, tq, tg, tk, tv, a);
    count_launch();
    if (e != cudaSuccess) return e;
  }
  {
    static std::atomic<unsigned long long> configured{0};
    if ((e = allow_dynamic_smem(dkv::attend_bwd_dkv_kernel, dkv::SMEM, configured)) != cudaSuccess) return e;
    e = launch_chained(dkv::attend_bwd_dkv_kernel, dim3((unsigned)((long long)a.n_slices * groups)), dim3(dkv::THREADS),
                       dkv::SMEM, st, tq, tg, tk, tv, a);
    count_launch();
  }
  return e;
}

}  // namespace dash
