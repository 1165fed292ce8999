// Stage 2, decode, on TMA + tcgen05 for sm_100a (Eq. 7 / Proposition 1; Algorithm 3; split-KV of Section 3.5).
//
// HBM-bound: per (batch, KV head) only the routed chunks' K and V rows are read, once, by bulk tensor
// copies into a 3-deep shared-memory ring (64 KiB per step = 128 KV tokens), so enough bytes are in flight
// to cover DRAM latency without occupying threads.  The arithmetic is tiny (g_q <= 16 query rows per KV
// head) and rides on the tensor cores in "transposed" form so that the KV tokens fill the MMA's M:
//     S^T[128 keys x 16 heads] = K_tile[128 x d] * Q^T[d x 16]          (heads padded to N = 16)
//     O^T[d = 128 x 16 heads] += V_tile^T[128 x 128 keys] * P^T[128 keys x 16]
// One softmax thread per key row (= TMEM lane of S^T); the per-head running maximum is shared through a
// small shared-memory reduction, the accumulator O^T is only 16 TMEM columns, so rescaling it is cheap.
// The routed list (plus the row's own, possibly partial, chunk) is cut into n_split contiguous ranges of
// 64-token sub-blocks, one thread block each; the block that sees the last arrival of its (batch, KV head)
// merges the partial (m, l, O) of all splits in split order (or, without a workspace, a separate merge kernel does).
// Every wait is bounded (DASH_ERR_TIMEOUT in the status word).
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace dash {

namespace {

constexpr int HD_MAX = 128;             // the shared-memory layout is the one of head_dim 128 (head_dim 64 fills half a tile)
constexpr int SUB = 64;                 // KV tokens per sub-block (one TMA box pair)
constexpr int STEP = 128;               // KV tokens per step = MMA M
constexpr int NST = 3;                  // K/V ring depth
constexpr int NH = 16;                  // heads padded to the MMA N
constexpr int DEC_THREADS = 192;
constexpr int MAX_RANGE = 512;          // sub-blocks one thread block can own
constexpr uint32_t TILE_BYTES = STEP * HD_MAX * 2;   // 32 KiB: two regions (d halves) of 128 rows x 128 B
constexpr uint32_t QT_BYTES = NH * HD_MAX * 2;       // 4 KiB: two regions of 16 rows x 128 B
constexpr uint32_t PT_BYTES = NH * STEP * 2;     // 4 KiB: two regions (key halves) of 16 rows x 128 B
constexpr uint32_t OFF_K = 0;
constexpr uint32_t OFF_V = OFF_K + NST * TILE_BYTES;
constexpr uint32_t OFF_QT = OFF_V + NST * TILE_BYTES;
constexpr uint32_t OFF_PT = OFF_QT + QT_BYTES;
constexpr uint32_t OFF_MISC = OFF_PT + PT_BYTES;
constexpr uint32_t TMEM_COLS = 64;      // S^T buffers at columns 0 and 16, O^T at 32
enum BarD { Q_READY = 0, S_FULL = 1, P_FULL = 3, P_EMPTY = 5, RED_BAR = 6, LRED_BAR = 8, K_FULL = 9, K_EMPTY = 9 + NST,
            V_FULL = 9 + 2 * NST, V_EMPTY = 9 + 3 * NST, N_BARS = 9 + 4 * NST };
// CPS = routed chunks per 64-token sub-block: 1 for chunks of 64 / 128 tokens, 2 / 4 for chunks of 32 / 16 (a
// sub-block then gathers that many chunks of the list, each fetched by its own TMA box and carrying its own bias).
template <int CPS>
struct MiscT {
  static constexpr int RANGE = MAX_RANGE / CPS;   // sub-blocks one thread block can own
  unsigned long long bar[N_BARS];
  uint32_t tmem_base;
  int abort_flag;
  float bias2[NST][2][CPS];
  int nvalid[NST][2];
  float red[2][4][NH];
  float lred[4][NH];
  int is_last;               // this block saw the last arrival of its (batch, KV head)
  int idx_s[RANGE][CPS];     // first KV token of each chunk slot of each owned sub-block (paged cache: inside its page)
  int pg_s[RANGE][CPS];      // outermost TMA coordinate of the slot: the sequence, or the physical page
  float bias_s[RANGE][CPS];
  int nval_s[RANGE];         // valid rows of the sub-block
};
constexpr size_t MISC_BYTES = sizeof(MiscT<1>) > sizeof(MiscT<2>)
                                  ? (sizeof(MiscT<1>) > sizeof(MiscT<4>) ? sizeof(MiscT<1>) : sizeof(MiscT<4>))
                                  : (sizeof(MiscT<2>) > sizeof(MiscT<4>) ? sizeof(MiscT<2>) : sizeof(MiscT<4>));
constexpr uint32_t DEC_SMEM = OFF_MISC + (uint32_t)MISC_BYTES;   // one size for every instantiation
static_assert(DEC_SMEM <= 232448, "shared memory budget");

struct DecodeArgs {
  Dims dm;
  int n_split;
  const int* kv_len;
  const int* count;
  const int* blk_idx;
  const float* blk_bias;
  const __nv_bfloat16* Q;
  float* partials;
  __nv_bfloat16* O;      // non-null: fused merge by the last split of each (batch, KV head)
  StatusBlock* sb;
};

__device__ __forceinline__ void tmem_ld16(uint32_t* r, uint32_t addr) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
               ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                 "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
               : "memory");
}

// head_dim 64 (HD = 64): K and V tiles are one 128-byte region per row.  S^T = K Q^T has four K steps.  The
// accumulator O^T would have only 64 rows, which is not an M = 128 shape, so the two 64-key sub-blocks of a step are
// stacked along M instead: A = [V_a^T ; V_b^T] (two MN blocks of 64, 8 KiB apart), K = 64 keys, B = [P_a^T | P_b^T]
// (N = 32): rows 0-63 / columns 0-15 hold V_a^T P_a^T and rows 64-127 / columns 16-31 hold V_b^T P_b^T (the other two
// quadrants are not used); the two are added when the partial is written.
template <int G, int CPS, int HD>
__global__ void __launch_bounds__(DEC_THREADS, 1)
decode_sm100_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, DecodeArgs a) {
  using MiscD = MiscT<CPS>;
  constexpr int W = SUB / CPS;          // rows of one chunk slot inside a sub-block
  extern __shared__ __align__(1024) uint8_t smem[];
  MiscD* misc = reinterpret_cast<MiscD*>(smem + OFF_MISC);
  const Dims& dm = a.dm;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t sbase = ptx::smem_u32(smem);
  auto bar = [&](int i) { return ptx::smem_u32(&misc->bar[i]); };
  volatile int* abort_flag = &misc->abort_flag;
  const int split = blockIdx.x, r = blockIdx.y, b = blockIdx.z;
  const int n_split = a.n_split;

  if (tid == 0) {
    misc->abort_flag = 0;
    if ((sbase & 1023u) != 0u) {
      report_error(a.sb, DASH_ERR_CUDA, 300);
      misc->abort_flag = 1;
    }
    ptx::mbar_init(bar(Q_READY), 128);
    ptx::mbar_init(bar(S_FULL), 1);
    ptx::mbar_init(bar(S_FULL + 1), 1);
    ptx::mbar_init(bar(P_FULL), 128);
    ptx::mbar_init(bar(P_FULL + 1), 128);
    ptx::mbar_init(bar(P_EMPTY), 1);
    ptx::mbar_init(bar(RED_BAR), 128);
    ptx::mbar_init(bar(RED_BAR + 1), 128);
    ptx::mbar_init(bar(LRED_BAR), 128);
    for (int s = 0; s < NST; ++s) {
      ptx::mbar_init(bar(K_FULL + s), 1);
      ptx::mbar_init(bar(K_EMPTY + s), 1);
      ptx::mbar_init(bar(V_FULL + s), 1);
      ptx::mbar_init(bar(V_EMPTY + s), 1);
    }
    ptx::fence_barrier_init();
  }
  if (warp == 5) {
    ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), TMEM_COLS);
    ptx::tmem_relinquish();
    ptx::tc_fence_before();
  }
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = misc->tmem_base;

  // barriers and tensor memory are set up; everything below reads what the routing kernels wrote
  int L = a.kv_len ? a.kv_len[b] : dm.seq_kv;   // the caller's input, not a product of the chain: read it before the wait
  chain_wait();
  chain_release();
  // an error already in the status word makes every role leave at its first wait (see the prefill kernel)
  if (a.sb && *reinterpret_cast<volatile int*>(&a.sb->status) != 0) *abort_flag = 1;
  __syncthreads();
  L = max(1, min(L, dm.seq_kv));
  const int c_own = (L - 1) / dm.B;
  const long long grp = (long long)b * dm.h_kv + r;
  const int spb = CPS > 1 ? 1 : dm.B / SUB;                     // sub-blocks per routed chunk (chunks >= 64 tokens)
  int n_routed = a.count[grp];
  DASH_CHECK(n_routed >= 0 && n_routed <= min(c_own, dm.T_s), a.sb, 310, n_routed = 0);
  const int n_routed_sub = CPS > 1 ? (n_routed + CPS - 1) / CPS : n_routed * spb;
  const int own_tokens = L - c_own * dm.B;                       // 1 .. B
  const int n_items = n_routed_sub + (own_tokens + SUB - 1) / SUB;
  const int per = (n_items + n_split - 1) / n_split;
  const int lo = min(n_items, split * per), hi = min(n_items, lo + per);
  const int n_own = hi - lo;                                     // <= MAX_RANGE by the host's choice of n_split
  const int n_steps = (n_own + 1) / 2;

  const long long loff = grp * dm.list_rows;

  if (warp == 4) {
    // ---------------- producer
    // owned sub-blocks -> (first token, bias, valid rows), staged once so the walk has no dependent global reads
    for (int k = lane; k < n_own; k += 32) {
      const int it = lo + k;
      if constexpr (CPS > 1) {
        if (it < n_routed_sub) {
          // CPS consecutive list entries; a short last group repeats its last chunk in rows that are marked invalid
          const int e0 = it * CPS, m = min(CPS, n_routed - e0);
#pragma unroll
          for (int s = 0; s < CPS; ++s) {
            const int e = e0 + min(s, m - 1);
            int cc = a.blk_idx[loff + e];
            DASH_CHECK(cc >= 0 && cc < c_own, a.sb, 311, cc = 0);
            kv_locate(dm, b, cc * dm.B, &misc->pg_s[k][s], &misc->idx_s[k][s]);
            DASH_CHECK(!dm.page_table || (unsigned)misc->pg_s[k][s] < (unsigned)dm.num_pages, a.sb, 313, misc->pg_s[k][s] = 0);
            misc->bias_s[k][s] = a.blk_bias[loff + e];
          }
          misc->nval_s[k] = m * dm.B;
        } else {
          // the own chunk (shorter than a sub-block): the rows behind it are fetched but marked invalid
#pragma unroll
          for (int s = 0; s < CPS; ++s) {
            kv_locate(dm, b, c_own * dm.B + s * W, &misc->pg_s[k][s], &misc->idx_s[k][s]);
            DASH_CHECK(!dm.page_table || (unsigned)misc->pg_s[k][s] < (unsigned)dm.num_pages, a.sb, 315, misc->pg_s[k][s] = 0);
            misc->bias_s[k][s] = 0.f;
          }
          misc->nval_s[k] = L - c_own * dm.B;
        }
        continue;
      }
      int tok0, nv;
      float bs;
      if (it < n_routed_sub) {
        const int e = it / spb, sub = it % spb;
        int cc = a.blk_idx[loff + e];
        DASH_CHECK(cc >= 0 && cc < c_own, a.sb, 312, cc = 0);
        tok0 = cc * dm.B + sub * SUB;
        bs = a.blk_bias[loff + e];
        nv = SUB;
      } else {
        const int sub = it - n_routed_sub;
        tok0 = c_own * dm.B + sub * SUB;
        bs = 0.f;
        nv = min(SUB, L - tok0);
      }
      kv_locate(dm, b, tok0, &misc->pg_s[k][0], &misc->idx_s[k][0]);
      DASH_CHECK(!dm.page_table || (unsigned)misc->pg_s[k][0] < (unsigned)dm.num_pages, a.sb, 314, misc->pg_s[k][0] = 0);
      misc->bias_s[k][0] = bs; misc->nval_s[k] = nv;
    }
    __syncwarp();
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmK);
      ptx::prefetch_tensormap(&tmV);
      bool ok = true;
      int s = 0, ph = 1;
      for (int j = 0; j < n_steps && ok; ++j) {
        const int k0 = 2 * j, k1 = (2 * j + 1 < n_own) ? 2 * j + 1 : 2 * j;   // an odd tail repeats its last sub-block
        // one 128-row tile: sub-blocks k0 and k1, each CPS boxes of W rows, for both halves of head_dim
        auto load_tile = [&](const CUtensorMap* tm, uint32_t dst, uint32_t barrier) {
          ptx::mbar_arrive_expect_tx(barrier, STEP * HD * 2);
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int k = h ? k1 : k0;
#pragma unroll
            for (int q = 0; q < CPS; ++q) {
              const int tok = misc->idx_s[k][q], pg = misc->pg_s[k][q];
              const uint32_t d = dst + (h * SUB + q * W) * 128;
              ptx::tma_load_4d(d, tm, barrier, 0, r, tok, pg);
              if constexpr (HD == 128) ptx::tma_load_4d(d + TILE_BYTES / 2, tm, barrier, 64, r, tok, pg);
            }
          }
        };
        ok = ptx::mbar_wait(bar(K_EMPTY + s), ph, abort_flag);
        if (!ok) break;
        load_tile(&tmK, sbase + OFF_K + s * TILE_BYTES, bar(K_FULL + s));
        ok = ptx::mbar_wait(bar(V_EMPTY + s), ph, abort_flag);
        if (!ok) break;
#pragma unroll
        for (int q = 0; q < CPS; ++q) {
          misc->bias2[s][0][q] = misc->bias_s[k0][q];
          misc->bias2[s][1][q] = misc->bias_s[k1][q];
        }
        misc->nvalid[s][0] = misc->nval_s[k0];
        misc->nvalid[s][1] = (k1 != k0) ? misc->nval_s[k1] : 0;
        load_tile(&tmV, sbase + OFF_V + s * TILE_BYTES, bar(V_FULL + s));
        if (++s == NST) { s = 0; ph ^= 1; }
      }
      if (!ok) {
        for (int q = 0; q < NST; ++q) {
          for (int k = 0; k < 200000 && !ptx::mbar_try_wait(bar(K_FULL + q), 0) && !ptx::mbar_try_wait(bar(K_FULL + q), 1); ++k) {}
          for (int k = 0; k < 200000 && !ptx::mbar_try_wait(bar(V_FULL + q), 0) && !ptx::mbar_try_wait(bar(V_FULL + q), 1); ++k) {}
        }
      }
    }
  } else if (warp == 5) {
    // ---------------- MMA issuer
    if (lane == 0 && n_steps > 0) {
      constexpr uint32_t IDESC_S = ptx::idesc_bf16_f32(128, NH, false, false);
      constexpr uint32_t IDESC_O = ptx::idesc_bf16_f32(128, HD == 128 ? NH : 2 * NH, true, false);
      const uint64_t kd0 = ptx::smem_desc_sw128(sbase + OFF_K, 16, 1024);
      const uint64_t qd0 = ptx::smem_desc_sw128(sbase + OFF_QT, 16, 1024);
      // MN-major A: the two MN blocks of 64 are the d halves, 16 KiB apart (head_dim 128), or the two 64-key
      // sub-blocks of the step, 8 KiB apart (head_dim 64)
      const uint64_t vd0 = ptx::smem_desc_sw128(sbase + OFF_V, HD == 128 ? TILE_BYTES / 2 : SUB * 128, 1024);
      const uint64_t pd0 = ptx::smem_desc_sw128(sbase + OFF_PT, 16, 1024);
      bool ok = ptx::mbar_wait(bar(Q_READY), 0, abort_flag);
      int ks = 0, kph = 0;
      auto issue_s = [&](int j) -> bool {
        if (!ptx::mbar_wait(bar(K_FULL + ks), kph, abort_flag)) return false;
        ptx::tc_fence_after();
        const uint64_t kd = kd0 + (uint64_t)((ks * TILE_BYTES) >> 4);
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          const uint64_t ad = kd + (uint64_t)(((k >> 2) * (TILE_BYTES / 2) + (k & 3) * 32) >> 4);
          const uint64_t bd = qd0 + (uint64_t)(((k >> 2) * (QT_BYTES / 2) + (k & 3) * 32) >> 4);
          ptx::mma_bf16_ss(tmem + (j & 1) * NH, ad, bd, IDESC_S, k > 0 ? 1u : 0u);
        }
        ptx::mma_commit(bar(S_FULL + (j & 1)));
        ptx::mma_commit(bar(K_EMPTY + ks));
        if (++ks == NST) { ks = 0; kph ^= 1; }
        return true;
      };
      if (ok) ok = issue_s(0);
      int vs = 0, vph = 0;
      for (int j = 0; j < n_steps && ok; ++j) {
        if (j + 1 < n_steps) ok = issue_s(j + 1);
        if (!ok) break;
        ok = ptx::mbar_wait(bar(V_FULL + vs), vph, abort_flag) && ptx::mbar_wait(bar(P_FULL + (j & 1)), (j >> 1) & 1, abort_flag);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint64_t vd = vd0 + (uint64_t)((vs * TILE_BYTES) >> 4);
#pragma unroll
        for (int k = 0; k < (HD == 128 ? STEP : SUB) / 16; ++k) {
          const uint64_t ad = vd + (uint64_t)((k * 16 * 128) >> 4);                                   // 16 key rows = 2048 B
          // head_dim 128: P^T is two K-major regions (key halves) of 16 rows; head_dim 64: the same bytes read as one
          // region of 32 rows (sub-block a's heads, then sub-block b's), 64 keys long
          const uint64_t bd = pd0 + (uint64_t)(((HD == 128 ? (k >> 2) * (PT_BYTES / 2) : 0) + (k & 3) * 32) >> 4);
          ptx::mma_bf16_ss(tmem + 2 * NH, ad, bd, IDESC_O, (j > 0 || k > 0) ? 1u : 0u);
        }
        ptx::mma_commit(bar(V_EMPTY + vs));
        ptx::mma_commit(bar(P_EMPTY));
        if (++vs == NST) { vs = 0; vph ^= 1; }
      }
    }
    __syncwarp();
  } else {
    // ---------------- softmax: thread = key row of the step = TMEM lane of S^T; also lane d of O^T
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    const float c1 = dm.sm_scale * 1.4426950408889634f;
    // Q^T tile: 16 rows (heads, zero beyond G) x 128 d, K-major, 128-byte swizzle; P^T rows beyond G stay zero
    for (int ch = tid; ch < NH * 16; ch += 128) {
      const int h = ch >> 4, c16 = ch & 15;            // 16-byte chunk c16 of head h: d = c16*8 .. +7
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (h < G && c16 * 8 < HD)
        v = *reinterpret_cast<const uint4*>(a.Q + (long long)b * dm.qs[0] + (long long)(r * G + h) * dm.qs[2] + c16 * 8);
      const uint32_t off = (c16 >> 3) * (QT_BYTES / 2) + h * 128 + (((c16 & 7) ^ (h & 7)) << 4);
      *reinterpret_cast<uint4*>(smem + OFF_QT + off) = v;
      *reinterpret_cast<uint4*>(smem + OFF_PT + off) = make_uint4(0u, 0u, 0u, 0u);
    }
    ptx::fence_proxy_async_smem();
    ptx::mbar_arrive(bar(Q_READY));

    float m[G], l[G];
#pragma unroll
    for (int h = 0; h < G; ++h) { m[h] = -INFINITY; l[h] = 0.f; }
    const int half = tid >> 6, row = tid & 63;
    bool ok = true;
    int vs = 0, vph = 0;
    for (int j = 0; j < n_steps && ok; ++j) {
      ok = ptx::mbar_wait(bar(V_FULL + vs), vph, abort_flag);     // step metadata visible, V tile landed
      if (!ok) break;
      const float b2 = misc->bias2[vs][half][CPS > 1 ? row / W : 0] * 1.4426950408889634f;
      const int nval = misc->nvalid[vs][half];
      const bool valid = row < nval;
      ok = ptx::mbar_wait(bar(S_FULL + (j & 1)), (j >> 1) & 1, abort_flag);
      if (!ok) break;
      ptx::tc_fence_after();
      uint32_t sr[16];
      tmem_ld16(sr, lane_addr + (j & 1) * NH);
      ptx::tmem_wait_ld();
      float x[G];
#pragma unroll
      for (int h = 0; h < G; ++h) {
        x[h] = valid ? fmaf(__uint_as_float(sr[h]), c1, b2) : -INFINITY;
        const float wm = warp_max(x[h]);
        if (lane == 0) misc->red[j & 1][warp][h] = wm;
      }
      // per-head maxima of the four warps meet through shared memory (bounded mbarrier, not bar.sync)
      ptx::mbar_arrive(bar(RED_BAR + (j & 1)));
      ok = ptx::mbar_wait(bar(RED_BAR + (j & 1)), (j >> 1) & 1, abort_flag);
      if (!ok) break;
      float corr[G];
      bool changed = false;
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const float ms = fmaxf(fmaxf(misc->red[j & 1][0][h], misc->red[j & 1][1][h]),
                               fmaxf(misc->red[j & 1][2][h], misc->red[j & 1][3][h]));
        const float mn = fmaxf(m[h], ms);
        changed |= mn > m[h];
        corr[h] = exp2f(m[h] - mn);     // 0 while nothing has been accumulated
        m[h] = mn;
      }
      __nv_bfloat16 pb[G];
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const float p = valid ? exp2f(x[h] - m[h]) : 0.f;
        l[h] = l[h] * corr[h] + p;
        pb[h] = __float2bfloat16_rn(p);
      }
      // the previous step's PV must be done before P^T is overwritten and before O^T is rescaled
      ok = ptx::mbar_wait(bar(P_EMPTY), (j & 1) ^ 1, abort_flag);
      if (!ok) break;
      ptx::tc_fence_after();
      if (j > 0 && changed) {
        // head_dim 64: this lane's live accumulator columns are h (sub-block a, lanes 0-63) or NH + h (lanes 64-127)
        const uint32_t o_addr = lane_addr + 2 * NH + ((HD == 64 && half) ? NH : 0);
        uint32_t o[16];
        tmem_ld16(o, o_addr);
        ptx::tmem_wait_ld();
#pragma unroll
        for (int h = 0; h < G; ++h) o[h] = __float_as_uint(__uint_as_float(o[h]) * corr[h]);
        tmem_st16(o_addr, o);
        ptx::tmem_wait_st();
      }
      // P^T[head h][key tid]: K-major rows of 64 keys, 128-byte swizzle
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const uint32_t off = half * (PT_BYTES / 2) + h * 128 + ((((row >> 3) & 7) ^ (h & 7)) << 4) + (row & 7) * 2;
        *reinterpret_cast<__nv_bfloat16*>(smem + OFF_PT + off) = pb[h];
      }
      // rows past the end of the sequence may hold anything (even NaN): zero their V rows, since 0 * NaN = NaN
      if (!valid && nval > 0 && nval < SUB) {
        uint8_t* vrow = smem + OFF_V + vs * TILE_BYTES + tid * 128;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          *reinterpret_cast<uint4*>(vrow + (q << 4)) = make_uint4(0u, 0u, 0u, 0u);
          *reinterpret_cast<uint4*>(vrow + TILE_BYTES / 2 + (q << 4)) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar(P_FULL + (j & 1)));
      if (++vs == NST) { vs = 0; vph ^= 1; }
    }

    // ---------------- partial (m, l, O) of this split
    if (ok && n_steps > 0) ok = ptx::mbar_wait(bar(P_EMPTY), (n_steps - 1) & 1, abort_flag);
    ptx::tc_fence_after();
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float ls = warp_sum(l[h]);
      if (lane == 0) misc->lred[warp][h] = ls;
    }
    ptx::mbar_arrive(bar(LRED_BAR));
    ok = ptx::mbar_wait(bar(LRED_BAR), 0, abort_flag) && ok;
    uint32_t o[16];
#pragma unroll
    for (int h = 0; h < 16; ++h) o[h] = 0u;
    if (ok && n_steps > 0) {
      tmem_ld16(o, lane_addr + 2 * NH + ((HD == 64 && (tid >> 6)) ? NH : 0));
      ptx::tmem_wait_ld();
    }
    if constexpr (HD == 64) {
      // O^T[d][h] = (sub-block a's part in lane d) + (sub-block b's part in lane 64 + d): the upper lanes hand theirs
      // over through the P^T tile, which no product reads any more
      float* comb = reinterpret_cast<float*>(smem + OFF_PT);       // [64][16]
      if (tid >= 64) {
#pragma unroll
        for (int h = 0; h < G; ++h) comb[(tid - 64) * NH + h] = __uint_as_float(o[h]);
      }
      ptx::mbar_arrive(bar(LRED_BAR));
      ok = ptx::mbar_wait(bar(LRED_BAR), 1, abort_flag) && ok;
      if (tid < 64) {
#pragma unroll
        for (int h = 0; h < G; ++h) o[h] = __float_as_uint(__uint_as_float(o[h]) + comb[tid * NH + h]);
      }
    }
    const long long pbase = (((long long)b * dm.h_q + (long long)r * G) * n_split + split) * (HD + 2);
#pragma unroll
    for (int h = 0; h < G; ++h) {
      float* pp = a.partials + pbase + (long long)h * n_split * (HD + 2);
      if (tid < HD) pp[2 + tid] = (n_steps > 0) ? __uint_as_float(o[h]) : 0.f;   // thread tid holds O^T[d = tid][h]
      if (tid == h) {
        pp[0] = (n_steps > 0) ? m[h] * 0.6931471805599453f : -INFINITY;   // the merge works in natural-log units
        pp[1] = misc->lred[0][h] + misc->lred[1][h] + misc->lred[2][h] + misc->lred[3][h];
      }
    }
    __threadfence();        // the partial is visible device-wide before this block counts itself as arrived
    ptx::tc_fence_before();
  }

  __syncthreads();
  if (warp == 5) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, TMEM_COLS);
  }
  if (a.O != nullptr) {
    // ---------------- the last split of this (batch, KV head) to arrive merges all of them, in split order
    int* counter = arrival_counters(a.sb) + grp;
    if (tid == 0) {
      const bool last = atomicAdd(counter, 1) == n_split - 1;
      if (last) *counter = 0;          // every split has arrived: the counter is ready for the next launch
      misc->is_last = last ? 1 : 0;
    }
    __syncthreads();
    if (misc->is_last) {
      __threadfence();
      constexpr int VPL = HD / 32;
      for (int h = warp; h < G; h += DEC_THREADS / 32) {
        const long long bh = (long long)b * dm.h_q + (long long)r * G + h;
        const float* p = a.partials + bh * n_split * (HD + 2);
        float M = -INFINITY;
        for (int s = 0; s < n_split; ++s) M = fmaxf(M, __ldcg(p + s * (HD + 2)));
        float Lsum = 0.f, acc[VPL];
#pragma unroll
        for (int v = 0; v < VPL; ++v) acc[v] = 0.f;
        for (int s = 0; s < n_split; ++s) {
          const float ms = __ldcg(p + s * (HD + 2));
          if (ms == -INFINITY) continue;
          const float w = __expf(ms - M);
          Lsum += w * __ldcg(p + s * (HD + 2) + 1);
          const float2* po = reinterpret_cast<const float2*>(p + s * (HD + 2) + 2 + lane * VPL);   // 8-byte aligned
          const float2 oa = __ldcg(po);
          acc[0] += w * oa.x; acc[1] += w * oa.y;
          if constexpr (VPL == 4) {
            const float2 ob = __ldcg(po + 1);
            acc[2] += w * ob.x; acc[3] += w * ob.y;
          }
        }
        const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
        __nv_bfloat16* op = a.O + (long long)b * dm.os[0] + (long long)(r * G + h) * dm.os[2] + lane * VPL;
#pragma unroll
        for (int v = 0; v < VPL; ++v) op[v] = __float2bfloat16_rn(acc[v] * inv);
      }
    }
  }
  if (tid == 0 && misc->abort_flag) report_error(a.sb, DASH_ERR_TIMEOUT, 301);
}

bool make_kv_map(CUtensorMap* out, const void* base, const Dims& dm, const long long* s) {
  // contiguous cache: [batch][seq_kv] tokens; paged cache: [num_pages][page_size]
  cuuint64_t dims[4] = {(cuuint64_t)dm.d, (cuuint64_t)dm.h_kv, (cuuint64_t)(dm.page_table ? dm.page_size : dm.seq_kv),
                        (cuuint64_t)(dm.page_table ? dm.num_pages : dm.batch)};
  auto st = [](long long e) { return (cuuint64_t)((e > 0 ? e : 8) * 2); };
  cuuint64_t strides[3] = {st(s[2]), st(s[1]), st(s[0])};
  cuuint32_t box[4] = {64u, 1u, (cuuint32_t)(dm.B < SUB ? dm.B : SUB), 1u};   // chunks below 64 tokens: one box per chunk
  return encode_bf16_sw128_4d(out, base, dims, strides, box);
}

}  // namespace

// Splits needed so that no thread block owns more than MAX_RANGE sub-blocks (0: shape not served here).
int decode_sm100_min_splits(const Dims& dm) {
  if (!dm.decode || dm.dtype != DASH_BF16 || (dm.d != 64 && dm.d != 128)) return 0;
  if (dm.B != 16 && dm.B != 32 && dm.B != 64 && dm.B != 128) return 0;
  if (dm.qs[2] % 8 != 0 || tensor_map_encoder() == nullptr) return 0;
  if (dm.B < SUB) {
    const int cps = SUB / dm.B, range = MAX_RANGE / cps;
    const int max_items = (dm.T_s + cps - 1) / cps + 1;
    return (max_items + range - 1) / range;
  }
  const int max_items = (dm.T_s + 1) * (dm.B / SUB);
  return (max_items + MAX_RANGE - 1) / MAX_RANGE;
}

cudaError_t launch_decode_sm100(const Dims& dm, int n_split, const void* Q, const void* K, const void* V,
                                const int* kv_len, const int* count, const int* blk_idx, const float* blk_bias,
                                float* partials, void* O, StatusBlock* sb, cudaStream_t st) {
  DecodeArgs a;
  a.O = (__nv_bfloat16*)O;
  a.dm = dm; a.n_split = n_split; a.kv_len = kv_len; a.count = count; a.blk_idx = blk_idx; a.blk_bias = blk_bias;
  a.Q = (const __nv_bfloat16*)Q; a.partials = partials; a.sb = sb;
  CUtensorMap tk, tv;
  if (!make_kv_map(&tk, K, dm, dm.ks) || !make_kv_map(&tv, V, dm, dm.vs)) return cudaErrorInvalidValue;
  dim3 grid(n_split, dm.h_kv, dm.batch);
  cudaError_t le = cudaSuccess;
#define DASH_DEC_HD(G, C, H)                                                                                    \
  {                                                                                                             \
    static std::atomic<unsigned long long> configured{0};                                                       \
    cudaError_t e = allow_dynamic_smem(decode_sm100_kernel<G, C, H>, DEC_SMEM, configured);                     \
    if (e != cudaSuccess) return e;                                                                             \
    le = launch_chained(decode_sm100_kernel<G, C, H>, grid, dim3(DEC_THREADS), DEC_SMEM, st, tk, tv, a);        \
  }
#define DASH_DEC_TC(G, C) \
  if (dm.d == 128) DASH_DEC_HD(G, C, 128) else DASH_DEC_HD(G, C, 64)
#define DASH_DEC_G(C)                                  \
  switch (dm.g_q) {                                    \
    case 1: DASH_DEC_TC(1, C); break;                  \
    case 2: DASH_DEC_TC(2, C); break;                  \
    case 4: DASH_DEC_TC(4, C); break;                  \
    case 8: DASH_DEC_TC(8, C); break;                  \
    case 16: DASH_DEC_TC(16, C); break;                \
    default: return cudaErrorInvalidValue;             \
  }
  if (dm.B >= SUB) { DASH_DEC_G(1) } else if (dm.B == 32) { DASH_DEC_G(2) } else { DASH_DEC_G(4) }
#undef DASH_DEC_G
#undef DASH_DEC_TC
#undef DASH_DEC_HD
  count_launch();
  return le;
}

}  // namespace dash
