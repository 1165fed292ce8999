// Stage 1 on tensor cores for sm_100a (Eq. 2, Eq. 4, Algorithm 2, Proposition 1), bf16 queries, head_dim 128 or 64.
//
// Tile = the (token, head-of-group) rows of TQ = min(128/g_q, chunk size) consecutive tokens of one (batch, KV head):
// 128 rows, or fewer live rows followed by zero-query padding when chunks are shorter than 128/g_q tokens;
// they share their candidate chunks.  The whole score tile X[128 rows][<= 512 chunks per block] is produced by
// tcgen05.mma into tensor memory and never leaves the SM (Algorithm 2 writes it to HBM).  The fp32
// summaries are split beforehand into three bf16 planes (hi + mid + lo = the fp32 value exactly), so that
// Q (exact in bf16) times the three planes, accumulated in fp32, carries fp32-class accuracy: the support
// must match a float64 evaluation except within 1e-4 of the threshold.
//
// A row is one TMEM lane.  Rows of up to 256 candidates have one solver thread each (two blocks per SM), so the
// threshold search needs no cross-thread reduction: up to 128 candidates are held in registers over all passes, longer
// rows stream out of tensor memory 32 columns at a time (loads software-pipelined over two register buffers).  Rows of
// more than 256 candidates (one block per SM) are split over three threads, whose partial sums meet in shared memory.
// tau is found by Newton's method (f convex and decreasing: monotone from below, finite for alpha = 2).
// The GQA group's heads sit in adjacent lanes; the group weights come from a halving shuffle exchange, one
// warp-synchronous step per 32 chunks; log w is parked in tensor memory until mu is known, then the compact
// bias lists are written.  Rows longer than one block's tensor memory are split over a thread-block cluster
// whose blocks all-reduce the per-row sums through distributed shared memory.  Waits are bounded as in the
// Stage 2 kernel.
#include <cuda.h>

#include <type_traits>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace dash {

namespace {

constexpr int SC = 64;               // candidate chunks per MMA block / staged summary tile
constexpr int HD_MAX = 128;          // the shared-memory layout is the one of head_dim 128; head_dim 64 fills half of each tile
// Solver threads per row.  Short rows (<= 256 candidates, two blocks per SM): one, the row lives in the thread.  Long
// rows (one block per SM holds up to 512 candidates of each row in tensor memory): three threads per row, in three
// warps that share a quarter of the TMEM lanes, each streaming a third of the row's columns, so that every
// scheduler of the SM has three solver warps to pick from instead of one; their partial sums meet through shared
// memory like those of the blocks of a cluster.  (Three, not four: 14 warps leave each thread 128 registers, which
// the streaming loops fill; 18 warps would leave 96 and spill.)
__host__ __device__ constexpr int split_of(int nst) { return nst == 1 ? 1 : 3; }
// MMA issuers: one for the short-row kernel (a single stage of summaries); two for long rows (even and odd 64-chunk
// blocks), fed by a three-stage ring of summary tiles: 192 products through one thread, each stage waiting a full L2
// round trip behind the product that freed it, take longer than the tensor pipe needs.
__host__ __device__ constexpr int issuers_of(int nst) { return nst == 1 ? 1 : 2; }
__host__ __device__ constexpr int sel_threads(int nst) { return (4 * split_of(nst) + 1 + issuers_of(nst)) * 32; }   // solver warps, producer, issuers
constexpr uint32_t Q_BYTES = 128 * HD_MAX * 2;        // 32 KiB
constexpr uint32_t PLANE_BYTES = SC * HD_MAX * 2;     // 16 KiB per plane per stage
constexpr uint32_t STAGE_BYTES = 3 * PLANE_BYTES;     // hi, mid, lo
constexpr int MAX_NEWTON = 64, MAX_NEWTON_GENERIC = 400;
constexpr int CLUSTER_COLS_FOR_BARRIERS = 512;     // = CLUSTER_COLS below: columns of one block's score tile

struct MiscS {
  unsigned long long bar[24];
  uint32_t tmem_base;
  int abort_flag;
};
// KB_*: up to three stages; XBAR: [warp 0..3][parity]; CB_DONE: one per 64-chunk block of the score tile (each completes
// exactly once, so a late waiter cannot mistake one completion for another)
enum BarS { Q_FULL = 0, X_FULL = 1, KB_FULL = 2, KB_EMPTY = 5, XBAR = 8, CB_DONE = 16 };
constexpr int MAX_CB = CLUSTER_COLS_FOR_BARRIERS / 64;
constexpr int CLUSTER_COLS = 512;      // candidates one block of a cluster holds in tensor memory
constexpr int MAX_CS = 4;              // widest cluster

template <int NST> struct SmemPlan {
  static constexpr uint32_t OFF_Q = 0;
  static constexpr uint32_t OFF_KB = Q_BYTES;
  static constexpr uint32_t OFF_XCH = OFF_KB + NST * STAGE_BYTES;
  // exchange slots [parity][participant][row] of (float, float); participants = cluster blocks x threads per row
  static constexpr uint32_t XCH_BYTES = NST == 1 ? 128u : 2u * MAX_CS * split_of(NST) * 128u * 16u;
  static constexpr uint32_t OFF_MISC = OFF_XCH + XCH_BYTES;
  static constexpr uint32_t TOTAL = OFF_MISC + sizeof(MiscS);
};

struct SelectTcArgs {
  Dims dm;
  int TQ, tile_base, n_tiles;   // tiles [tile_base, tile_base + n_tiles) of every (batch, KV head) are handled here
  uint32_t tmem_cols;     // power of two >= 32 covering the widest tile
  long long plane_rows;   // rows of one bf16 plane = batch * h_kv * T_s
  uint32_t* mask;
  int* count;
  int* blk_idx;
  float* blk_bias;
  float* tau;
  StatusBlock* sb;
};

__global__ void kbar_split_kernel(const float* __restrict__ kbar, __nv_bfloat16* __restrict__ planes, long long n) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  chain_wait();
  chain_release();
  if (i >= n) return;
  const float x = kbar[i];
  const __nv_bfloat16 hi = __float2bfloat16_rn(x);
  const float r1 = x - __bfloat162float(hi);
  const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
  const float r2 = r1 - __bfloat162float(mid);
  planes[i] = hi;
  planes[n + i] = mid;
  planes[2 * n + i] = __float2bfloat16_rn(r2);
}

// SHORT: the tile has fewer than 128 live rows (chunks shorter than 128 / g_q tokens); full tiles compile without
// any of the padding-row handling.
template <int NST, int G, int CS, int HD, bool SHORT>
__global__ void __launch_bounds__(sel_threads(NST), NST == 1 ? 2 : 1)
select_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKB, SelectTcArgs a) {
  using SP = SmemPlan<NST>;
  extern __shared__ __align__(1024) uint8_t smem[];
  MiscS* misc = reinterpret_cast<MiscS*>(smem + SP::OFF_MISC);
  constexpr int SPLIT = split_of(NST), NSOLVE = 4 * SPLIT, W_PROD = NSOLVE, W_MMA = NSOLVE + 1;
  constexpr int N_ISSUE = issuers_of(NST);      // issuing warps W_MMA .. W_MMA + N_ISSUE - 1; the first owns the TMEM allocation
  constexpr int SEL_TC_THREADS = sel_threads(NST);
  const Dims& dm = a.dm;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t sbase = ptx::smem_u32(smem);
  auto bar = [&](int i) { return ptx::smem_u32(&misc->bar[i]); };
  volatile int* abort_flag = &misc->abort_flag;

  // A cluster of CS blocks shares one tile: block `cr` holds candidates [cr*512, cr*512 + 512) of all 128 rows
  // and the per-row partial sums meet through distributed shared memory (CS = 1: a plain block).
  const int cr = CS > 1 ? (int)ptx::cluster_ctarank() : 0;
  const int cid = (int)(blockIdx.x / CS);
  const int groups = dm.batch * dm.h_kv;
  const int tile = a.tile_base + a.n_tiles - 1 - cid / groups;
  const int grp = cid % groups;
  const int b = grp / dm.h_kv, r = grp % dm.h_kv;
  const int TQ = a.TQ;
  constexpr int g_q = G;
  const int i0 = tile * TQ;
  const int c_own = i0 / dm.B;
  // candidates of the tile's rows; with a local window its chunks are not scored (window_rows_kernel lists them)
  const int n_cand = min(max(c_own - dm.local_blocks, 0), dm.T_s);   // (c_own <= T_s in a prefill)
  constexpr int CCOLS = CLUSTER_COLS;
  const int c_lo = cr * CCOLS;                                 // first candidate this block holds
  const int n_loc = CS > 1 ? max(0, min(CCOLS, n_cand - c_lo)) : n_cand;
  const int n_blk = (n_loc + SC - 1) / SC;

  if (tid == 0) {
    misc->abort_flag = 0;
    if ((sbase & 1023u) != 0u) {
      report_error(a.sb, DASH_ERR_CUDA, 200);
      misc->abort_flag = 1;
    }
    ptx::mbar_init(bar(Q_FULL), 1);
    ptx::mbar_init(bar(X_FULL), N_ISSUE);
    for (int s = 0; s < NST; ++s) {
      ptx::mbar_init(bar(KB_FULL + s), 1);
      ptx::mbar_init(bar(KB_EMPTY + s), 1);
    }
    for (int s = 0; s < 8; ++s) ptx::mbar_init(bar(XBAR + s), CS * SPLIT * 32);
    for (int s = 0; s < MAX_CB; ++s) ptx::mbar_init(bar(CB_DONE + s), 1);
    ptx::fence_barrier_init();
  }
  if (warp == W_MMA) {
    ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), a.tmem_cols);
    ptx::tmem_relinquish();
    ptx::tc_fence_before();
  }
  // Rows of the Q tile beyond its TQ * g_q live rows (chunks shorter than 128 / g_q tokens) are never written by the
  // TMA box: zero queries give zero logits, and nothing those rows compute is stored.
  if constexpr (SHORT) {
    const int first = TQ * g_q * 8;                 // 16-byte pieces before the first dead row (a row is 128 bytes)
    for (int regn = 0; regn < HD / 64; ++regn)
      for (int k = first + tid; k < 128 * 8; k += SEL_TC_THREADS)
        *reinterpret_cast<uint4*>(smem + SP::OFF_Q + regn * (Q_BYTES / 2) + k * 16) = make_uint4(0u, 0u, 0u, 0u);
    ptx::fence_proxy_async_smem();
  }
  __syncthreads();
  if (CS > 1) ptx::cluster_sync_all();     // every block's barriers exist before anybody arrives on them remotely
  ptx::tc_fence_after();
  const uint32_t tmem = misc->tmem_base;
  // barriers and tensor memory are set up; from here on the kernel reads the planes the previous kernel wrote
  chain_wait();
  chain_release();
  // an error already in the status word (a wait that ran out in an earlier block or kernel) makes every role
  // leave at its first wait, so the rest of the grid retires in microseconds instead of a wait limit per block
  if (a.sb && *reinterpret_cast<volatile int*>(&a.sb->status) != 0) *abort_flag = 1;
  __syncthreads();

  if (warp == W_PROD) {
    // ---------------- producer: Q tile, then the three planes of every 64-chunk block of summaries
    if (lane == 0 && n_loc > 0) {
      ptx::prefetch_tensormap(&tmQ);
      ptx::prefetch_tensormap(&tmKB);
      ptx::mbar_arrive_expect_tx(bar(Q_FULL), SHORT ? (uint32_t)(TQ * g_q * HD * 2) : 128 * HD * 2);   // the box holds the live rows
      ptx::tma_load_4d(sbase + SP::OFF_Q, &tmQ, bar(Q_FULL), 0, r * g_q, i0, b);
      if constexpr (HD == 128) ptx::tma_load_4d(sbase + SP::OFF_Q + Q_BYTES / 2, &tmQ, bar(Q_FULL), 64, r * g_q, i0, b);
      const long long row0 = ((long long)b * dm.h_kv + r) * dm.T_s + c_lo;
      bool ok = true;
      for (int cb = 0; cb < n_blk && ok; ++cb) {
        const int s = cb % NST;
        ok = ptx::mbar_wait(bar(KB_EMPTY + s), ((cb / NST) & 1) ^ 1, abort_flag);
        if (!ok) break;
        ptx::mbar_arrive_expect_tx(bar(KB_FULL + s), 3 * SC * HD * 2);
        for (int pl = 0; pl < 3; ++pl) {
          const uint32_t dst = sbase + SP::OFF_KB + s * STAGE_BYTES + pl * PLANE_BYTES;
          const int row = (int)(pl * a.plane_rows + row0 + (long long)cb * SC);
          ptx::tma_load_4d(dst, &tmKB, bar(KB_FULL + s), 0, row, 0, 0);
          if constexpr (HD == 128) ptx::tma_load_4d(dst + PLANE_BYTES / 2, &tmKB, bar(KB_FULL + s), 64, row, 0, 0);
        }
      }
      if (!ok) {
        for (int s = 0; s < NST; ++s)
          for (int k = 0; k < 200000 && !ptx::mbar_try_wait(bar(KB_FULL + s), 0) && !ptx::mbar_try_wait(bar(KB_FULL + s), 1); ++k) {}
      }
    }
  } else if (warp >= W_MMA) {
    // ---------------- MMA issuers: X[:, cb*64 .. +64) = Q Kbar_hi^T + Q Kbar_mid^T + Q Kbar_lo^T; with two issuers,
    // issuer k takes the blocks cb = k, k + 2, ...  Every issuer waits for EVERY block's tile, also those it leaves to
    // the other one: a parity wait only tells a phase from its neighbour, so a thread must see a barrier's phases in
    // order (an issuer that skipped a phase could take the stage's previous fill for the one it waits for).
    if (lane == 0 && n_loc > 0) {
      constexpr uint32_t IDESC = ptx::idesc_bf16_f32(128, SC, false, false);
      bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag);
      for (int cb = 0; cb < n_blk && ok; ++cb) {
        const int s = cb % NST;
        ok = ptx::mbar_wait(bar(KB_FULL + s), (cb / NST) & 1, abort_flag);
        if (!ok) break;
        if (cb % N_ISSUE != warp - W_MMA) continue;
        ptx::tc_fence_after();
        // descriptors differ only in the start-address field (16-byte units, no carry into the next field): built once
        // per stage, then one add per MMA keeps the issuing thread's instruction stream short
        const uint64_t qd0 = ptx::smem_desc_sw128(sbase + SP::OFF_Q, 16, 1024);
        const uint64_t kd0 = ptx::smem_desc_sw128(sbase + SP::OFF_KB + s * STAGE_BYTES, 16, 1024);
#pragma unroll
        for (int pl = 0; pl < 3; ++pl) {
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) {
            const uint64_t ad = qd0 + (uint64_t)(((k >> 2) * (Q_BYTES / 2) + (k & 3) * 32) >> 4);
            const uint64_t bd = kd0 + (uint64_t)((pl * PLANE_BYTES + (k >> 2) * (PLANE_BYTES / 2) + (k & 3) * 32) >> 4);
            ptx::mma_bf16_ss(tmem + cb * SC, ad, bd, IDESC, (pl > 0 || k > 0) ? 1u : 0u);
          }
        }
        ptx::mma_commit(bar(KB_EMPTY + s));
        ptx::mma_commit(bar(CB_DONE + cb));
      }
      if (ok) ptx::mma_commit(bar(X_FULL));
    }
    __syncwarp();
  } else {
    // ---------------- solver: row = TMEM lane; SPLIT threads per row (warps q, q + 4, ...: the same quarter of the
    // lanes), thread `part` of a row owning a contiguous share of the row's 32-column chunks
    const int q4 = SPLIT == 1 ? warp : (warp & 3), part = SPLIT == 1 ? 0 : (warp >> 2);
    const int m = q4 * 32 + lane;
    const int t = m / g_q, hh = m % g_q;
    const int i = i0 + t;
    const bool row_valid = SHORT ? (i < dm.seq_q && t < TQ) : i < dm.seq_q;   // (a short tile ends with zero-query rows)
    const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
    const int e_int = dm.e_int;
    const float e = dm.e, xs = dm.x_scale;
    const int n_chunks = (n_loc + 31) / 32;
    const int per_part = (n_chunks + SPLIT - 1) / SPLIT;
    const int k_lo = SPLIT == 1 ? 0 : min(part * per_part, n_chunks);                  // this thread's chunks
    const int k_hi = SPLIT == 1 ? n_chunks : min(k_lo + per_part, n_chunks);
    bool ok = true;
    float tau = 0.f;
    // rows that are held in registers wait for the whole score tile here; streamed rows start on the tile's first
    // 64-chunk blocks while the later ones are still being produced (see solve_streaming)
    const bool row_in_regs = CS == 1 && SPLIT == 1 && n_chunks <= 4;
    if (n_loc > 0 && (row_in_regs || n_cand == 0)) {
      ok = ptx::mbar_wait(bar(X_FULL), 0, abort_flag);
      ptx::tc_fence_after();
    }
    // Cluster all-reduce of two floats per row: every thread writes its pair into slot [parity][its rank][row]
    // of every block, arrives (release, cluster scope) on every block's per-warp barrier, waits on its own and
    // reads the CS pairs back in rank order, so all blocks see bit-identical results and take the same branches.
    // The participants of a row are ordered by the candidates they hold: rank = cluster rank * SPLIT + part.
    constexpr int NP = CS * SPLIT;
    const int my_rank = cr * SPLIT + part;
    int xround = 0;
    // what a round leaves behind: sums of both values over all participants (added in rank order, so every
    // participant holds the same bits and takes the same branches), the maximum of the first, and the sum of the
    // first over the participants ranked below this one
    float x_sum_a = 0.f, x_sum_b = 0.f, x_sum_c = 0.f, x_max_a = 0.f, x_below_a = 0.f;
    auto exchange = [&](float va, float vb, float vc = 0.f) -> bool {
      if constexpr (NP == 1) {
        x_sum_a = x_max_a = va; x_sum_b = vb; x_sum_c = vc; x_below_a = 0.f;
        return true;
      } else {
        const int par = xround & 1;
        float4* xbuf = reinterpret_cast<float4*>(smem + SP::OFF_XCH);          // [2][NP][128]
        float4* mine = &xbuf[(par * NP + my_rank) * 128 + m];
        const uint32_t mybar = bar(XBAR + q4 * 2 + par);
        if constexpr (CS == 1) {
          *mine = make_float4(va, vb, vc, 0.f);
          ptx::mbar_arrive(mybar);
          if (!ptx::mbar_wait(mybar, (xround >> 1) & 1, abort_flag)) return false;
        } else {
          const uint32_t slot = ptx::smem_u32(mine);
#pragma unroll
          for (int pr = 0; pr < CS; ++pr) ptx::st_cluster_f32x4(ptx::map_to_rank(slot, pr), va, vb, vc, 0.f);
#pragma unroll
          for (int pr = 0; pr < CS; ++pr) ptx::mbar_arrive_cluster(ptx::map_to_rank(mybar, pr));
          if (!ptx::mbar_wait_cluster(mybar, (xround >> 1) & 1, abort_flag)) return false;
        }
        float sa = 0.f, sb = 0.f, sc = 0.f, mxa = -INFINITY, below = 0.f;
#pragma unroll
        for (int pr = 0; pr < NP; ++pr) {
          const float4 v = xbuf[(par * NP + pr) * 128 + m];
          sa += v.x; sb += v.y; sc += v.z;
          mxa = fmaxf(mxa, v.x);
          if (pr < my_rank) below += v.x;
        }
        x_sum_a = sa; x_sum_b = sb; x_sum_c = sc; x_max_a = mxa; x_below_a = below;
        ++xround;
        return true;
      }
    };
    auto xsum_a = [&]() { return x_sum_a; };
    auto xsum_b = [&]() { return x_sum_b; };
    // Newton on f(tau) = sum [x - tau]_+^e - 1 (steps taken on f^(1/e), see newton_delta), convex and decreasing.
    // From the left of the root the iterates rise monotonically and never pass it; from the right one step lands
    // on the left.  The start is the root
    // of the same equation with every candidate taken as active (closed form for alpha = 2 and 1.5), clamped to
    // max - 1 <= tau* < max, which saves the slow first halvings of a start at max - 1.
    // The body below runs with the exponent as a compile-time constant for alpha = 1.5 (integer power 2, the
    // paper's setting): the per-candidate loops then hold no tests of it.  Other exponents take the same code
    // with the run-time value.
    auto solve = [&](auto ei_tag) {
    constexpr int EI_STATIC = decltype(ei_tag)::value;
    const int ei = EI_STATIC >= 0 ? EI_STATIC : e_int;
    const int max_it = ei ? MAX_NEWTON : MAX_NEWTON_GENERIC;
    auto start_tau = [&](float mx, float s1, float s2) -> float {   // s1, s2: sums of (x - mx), (x - mx)^2
      const float n = (float)n_cand;
      float t = -1.f;
      if (ei == 1) {
        t = (s1 - 1.f) / n;
      } else if (ei == 2) {
        const float mean = s1 / n, ss = s2 - s1 * mean;      // ss = sum of (x - mean)^2
        if (ss < 1.f) t = mean - sqrtf((1.f - ss) / n);
        // A second guess from the row's first two moments alone: were the candidates normal with that mean and
        // deviation s, n E[(x - tau)_+^2] = 1 would read G(z) = 1 / ss with z = (tau - mean) / s and
        // G(z) = (1 + z^2) Q(z) - z phi(z); z(ln G) is smooth, a quartic holds it within 0.07 over G in [1e-7, 3].
        // It lands near the root where the all-active guess, a lower bound, sits far below it (sparse supports);
        // the larger of the two is taken.  Either side of the root is a valid start (see above), so a row that is
        // far from normal costs a pass at worst.
        if (n_cand >= 8 && ss > 0.f) {
          const float L = -__logf(fminf(fmaxf(ss, 0.3334f), 1e7f));
          const float z = fmaf(fmaf(fmaf(fmaf(-8.93074e-05f, L, -0.0037117f), L, -0.0612527f), L, -0.717421f), L, -0.499476f);
          t = fmaxf(t, fmaf(z, sqrtf(ss / n), mean));
        }
      }
      return mx + fminf(fmaxf(t, -1.f), -1e-6f);
    };
    auto newton_step = [&](float f, float g, bool& done) {
      if (done) return;
      if (fabsf(f - 1.f) <= NEWTON_F_TOL || !(g > 0.f)) { done = true; return; }
      const float nt = tau + newton_delta(f, g, ei, e);
      if (nt == tau) done = true; else tau = nt;
    };
    constexpr bool CAN_HOLD = CS == 1 && SPLIT == 1;   // one thread per row: a short row can live in its registers
    float xr[CAN_HOLD ? 4 : 1][32];                // the whole row, when it has at most 128 candidates
    const bool in_regs = CAN_HOLD && n_chunks <= 4;
    auto solve_in_regs = [&]() {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (k < n_chunks) {
          uint32_t v[32];
          DASH_TMEM_LD32(v, lane_addr + k * 32);
          ptx::tmem_wait_ld();
          const int lim = n_cand - k * 32;
#pragma unroll
          for (int c = 0; c < 32; ++c) xr[k][c] = c < lim ? __uint_as_float(v[c]) * xs : -INFINITY;
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) xr[k][c] = -INFINITY;
        }
      }
      // several independent chains per reduction: one chain of 128 dependent operations would cost its latency 128 times
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int c = 0; c < 32; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], xr[k][c]);
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      float2 s1v[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)}, s2v[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      const float2 nmx = make_float2(-mx, -mx);
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          float2 y = __fadd2_rn(make_float2(xr[k][c], xr[k][c + 1]), nmx);     // two candidates per instruction
          y.x = xr[k][c] > -INFINITY ? y.x : 0.f;
          y.y = xr[k][c + 1] > -INFINITY ? y.y : 0.f;
          s1v[(c >> 1) & 1] = __fadd2_rn(s1v[(c >> 1) & 1], y);
          s2v[(c >> 1) & 1] = __ffma2_rn(y, y, s2v[(c >> 1) & 1]);
        }
      const float s1 = (s1v[0].x + s1v[0].y) + (s1v[1].x + s1v[1].y);
      const float s2 = (s2v[0].x + s2v[0].y) + (s2v[1].x + s2v[1].y);
      tau = start_tau(mx, s1, s2);
      bool done = false;
      for (int it = 0; it < max_it; ++it) {
        float f[4] = {0.f, 0.f, 0.f, 0.f}, g[4] = {0.f, 0.f, 0.f, 0.f};
        if constexpr (EI_STATIC == 2) {
          // alpha = 1.5: F += m^2, G += m, two candidates per packed instruction, four chains of pairs
          float2 fv[4], gv[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) fv[q] = gv[q] = make_float2(0.f, 0.f);
          const float2 ntau = make_float2(-tau, -tau);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            if (k < n_chunks) {
#pragma unroll
              for (int c = 0; c < 32; c += 2) {
                float2 mm = __fadd2_rn(make_float2(xr[k][c], xr[k][c + 1]), ntau);
                mm.x = fmaxf(mm.x, 0.f);
                mm.y = fmaxf(mm.y, 0.f);
                fv[(c >> 1) & 3] = __ffma2_rn(mm, mm, fv[(c >> 1) & 3]);
                gv[(c >> 1) & 3] = __fadd2_rn(gv[(c >> 1) & 3], mm);
              }
            }
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) { f[q] = fv[q].x + fv[q].y; g[q] = gv[q].x + gv[q].y; }
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            if (k < n_chunks) {
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                const float mm = fmaxf(xr[k][c] - tau, 0.f);
                f[c & 3] += pow_e(mm, ei, e);
                g[c & 3] += pow_em1(mm, ei, e);
              }
            }
          }
        }
        newton_step((f[0] + f[1]) + (f[2] + f[3]), (g[0] + g[1]) + (g[2] + g[3]), done);
        if (__all_sync(0xffffffffu, done)) break;
      }
    };
    auto solve_streaming = [&]() {
      // longer rows stream from tensor memory every pass (and, in a cluster, meet the other blocks' partial sums).
      // The 32-column loads are software-pipelined over two register buffers: with one block per SM a solver
      // warp has its scheduler to itself, so an exposed load latency per chunk would be pure idle time.
      auto stream = [&](auto&& body) {
        if (k_lo >= k_hi) return;                  // a row shorter than the threads it is split over
        uint32_t va[32], vb[32];
        DASH_TMEM_LD32(va, lane_addr + k_lo * 32);
        for (int k = k_lo; k < k_hi; k += 2) {
          DASH_TMEM_WAIT_LD32(va);
          if (k + 1 < k_hi) DASH_TMEM_LD32(vb, lane_addr + (k + 1) * 32);
          body(va, k);
          if (k + 1 < k_hi) {
            DASH_TMEM_WAIT_LD32(vb);
            if (k + 2 < k_hi) DASH_TMEM_LD32(va, lane_addr + (k + 2) * 32);
            body(vb, k + 1);
          }
        }
      };
      // columns past the row's last candidate (only in the last chunk) hold scores of later chunks: -inf them
      auto cut_tail = [&](uint32_t (&v)[32], int k) {
        const int lim = n_loc - k * 32;
        if (lim < 32) {
#pragma unroll
          for (int c = 0; c < 32; ++c) v[c] = c < lim ? v[c] : 0xff800000u;
        }
      };
      // First pass, while the tile is still being produced: a 32-column chunk is read as soon as its 64-chunk block is
      // complete (CB_DONE), and gives the row's maximum and the raw moments sum x, sum x^2 in one sweep; the moments
      // about the maximum, which the start value needs, follow from them after the one exchange.
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      float s1v[4] = {0.f, 0.f, 0.f, 0.f}, s2v[4] = {0.f, 0.f, 0.f, 0.f};
      for (int k = k_lo; k < k_hi && ok; ++k) {
        ok = ptx::mbar_wait(bar(CB_DONE + (k >> 1)), 0, abort_flag);
        if (!ok) break;
        ptx::tc_fence_after();
        uint32_t v[32];
        DASH_TMEM_LD32(v, lane_addr + k * 32);
        ptx::tmem_wait_ld();
        const int lim = n_loc - k * 32;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          if (c < lim) {
            const float y = __uint_as_float(v[c]) * xs;
            mx4[c & 3] = fmaxf(mx4[c & 3], y);
            s1v[c & 3] += y;
            s2v[c & 3] = fmaf(y, y, s2v[c & 3]);
          }
        }
      }
      // the later passes read all of this thread's columns at will: the whole tile must be there
      if (ok && n_loc > 0) {
        ok = ptx::mbar_wait(bar(X_FULL), 0, abort_flag);
        ptx::tc_fence_after();
      }
      float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      ok = ok && exchange(mx, (s1v[0] + s1v[1]) + (s1v[2] + s1v[3]), (s2v[0] + s2v[1]) + (s2v[2] + s2v[3]));
      mx = x_max_a;
      {
        // sum (x - mx) = S1 - n mx,  sum (x - mx)^2 = S2 - 2 mx S1 + n mx^2  (only the start value depends on them)
        const float n = (float)n_cand, S1 = x_sum_b, S2 = x_sum_c;
        tau = start_tau(mx, S1 - n * mx, fmaxf(fmaf(n * mx, mx, fmaf(-2.f * mx, S1, S2)), 0.f));
      }
      bool done = false;
      for (int it = 0; it < max_it && ok; ++it) {
        float f[4] = {0.f, 0.f, 0.f, 0.f}, g[4] = {0.f, 0.f, 0.f, 0.f};
        if constexpr (EI_STATIC == 2) {
          // alpha = 1.5: two candidates per packed instruction (scale and shift, F += m^2, G += m)
          float2 fv[4], gv[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) fv[q] = gv[q] = make_float2(0.f, 0.f);
          const float2 xs2 = make_float2(xs, xs), ntau = make_float2(-tau, -tau);
          stream([&](uint32_t (&v)[32], int k) {
            cut_tail(v, k);               // -inf * xs - tau = -inf: contributes nothing
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              float2 mm = __ffma2_rn(make_float2(__uint_as_float(v[c]), __uint_as_float(v[c + 1])), xs2, ntau);
              mm.x = fmaxf(mm.x, 0.f);
              mm.y = fmaxf(mm.y, 0.f);
              fv[(c >> 1) & 3] = __ffma2_rn(mm, mm, fv[(c >> 1) & 3]);
              gv[(c >> 1) & 3] = __fadd2_rn(gv[(c >> 1) & 3], mm);
            }
          });
#pragma unroll
          for (int q = 0; q < 4; ++q) { f[q] = fv[q].x + fv[q].y; g[q] = gv[q].x + gv[q].y; }
        } else {
          stream([&](uint32_t (&v)[32], int k) {
            cut_tail(v, k);               // -inf * xs - tau = -inf: contributes nothing
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const float mm = fmaxf(fmaf(__uint_as_float(v[c]), xs, -tau), 0.f);
              f[c & 3] += pow_e(mm, ei, e);
              g[c & 3] += pow_em1(mm, ei, e);
            }
          });
        }
        ok = exchange((f[0] + f[1]) + (f[2] + f[3]), (g[0] + g[1]) + (g[2] + g[3]));
        if (!ok) break;
        newton_step(xsum_a(), xsum_b(), done);
        if (__all_sync(0xffffffffu, done)) break;
      }
    };
    if constexpr (CAN_HOLD) {
      if (ok && n_cand > 0 && in_regs) solve_in_regs();
      else if (ok && n_cand > 0) solve_streaming();
    } else {
      if (ok && n_cand > 0) solve_streaming();
    }
    if (ok && row_valid && a.tau && my_rank == 0) a.tau[((long long)b * dm.h_q + r * g_q + hh) * dm.seq_q + i] = tau;

    // ---------------- group weights, mask words, log w, compact lists
    // The g_q heads of a token sit in g_q adjacent lanes.  Per 32-chunk step every lane raises its own margins
    // to the power e and the group sums them with a halving exchange (log2(g_q) rounds of shuffles), after
    // which lane j of the group owns the sums of 32/g_q contiguous chunks: w = sum / g_q, bit = (sum > 0),
    // log w = log(sum) - log(g_q).  log w (or +inf) is parked in the lane's own TMEM columns (the scores there
    // are spent), so the second sweep, which needs mu = mean log w, writes the final biases straight into the
    // compact list: no read-modify-write of global memory.
    constexpr int OWN = 32 / G;                                  // chunks a lane owns per step
    const int own0 = [&] {                                       // first owned chunk: bit k of hh picks a half
      int base = 0, width = 32;
#pragma unroll
      for (int o = 1; o < G; o <<= 1) { width >>= 1; if (hh & o) base += width; }
      return base;
    }();
    const long long row_id = ((long long)b * dm.h_kv + r) * dm.seq_q + i;
    const long long loff = ((long long)b * dm.h_kv + r) * dm.list_rows + list_row_offset(dm, min(i, dm.seq_q - 1));
    uint32_t* mrow = a.mask + row_id * dm.W;
    const float log_gq = logf((float)G);
    float slog = 0.f;
    int nsel = 0;
    auto group_sums = [&](float (&pe)[32]) {
      // after the call pe[0 .. OWN) hold the group sums of chunks own0 .. own0+OWN
      int live = 32;
#pragma unroll
      for (int o = 1; o < G; o <<= 1) {
        const bool upper = (hh & o) != 0;
        const int half = live / 2;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          if (c < half) {
            const float mine = upper ? pe[c + half] : pe[c];
            const float give = upper ? pe[c] : pe[c + half];
            pe[c] = mine + __shfl_xor_sync(0xffffffffu, give, o);
          }
        }
        live = half;
      }
    };
    if (ok) {
      // one 32-chunk step: pe holds this lane's [x - tau]_+^e on entry and is consumed
      auto chunk_step = [&](int k, float (&pe)[32]) {
        group_sums(pe);
        uint32_t bits = 0;
        uint32_t lwv[OWN];
#pragma unroll
        for (int c = 0; c < OWN; ++c) lwv[c] = 0x7f800000u;       // +inf: not routed
#pragma unroll
        for (int q = 0; q < OWN; ++q) {
          if (pe[q] > 0.f) {
            const float lw = __logf(pe[q]) - log_gq;
            lwv[q] = __float_as_uint(lw);
            slog += lw;
            bits |= 1u << (own0 + q);
          }
        }
#pragma unroll
        for (int o = 1; o < G; o <<= 1) bits |= __shfl_xor_sync(0xffffffffu, bits, o);
        ptx::tmem_st_n<OWN>(lane_addr + k * 32, lwv);            // slot q of this lane = chunk own0 + q of step k
        if (row_valid && hh == 0) {
          const int wj = cr * (CCOLS / 32) + k;                // mask word of this step
          mrow[wj] = bits | (((c_own >> 5) == wj) ? (1u << (c_own & 31)) : 0u);
        }
        nsel += __popc(bits);
      };
      if (in_regs) {
        // the register-resident row is spent after this sweep: raise it to the power in place, no second copy
        if constexpr (CAN_HOLD) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (k < n_chunks) {
#pragma unroll
            for (int c = 0; c < 32; ++c) xr[k][c] = pow_e(fmaxf(xr[k][c] - tau, 0.f), ei, e);
            chunk_step(k, xr[k]);
          }
        }
        }
      } else {
        for (int k = k_lo; k < k_hi; ++k) {
          float pe[32];
          uint32_t v[32];
          DASH_TMEM_LD32(v, lane_addr + k * 32);
          ptx::tmem_wait_ld();
          const int lim = n_loc - k * 32;
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const float mm = fmaxf(fmaf(__uint_as_float(v[c]), xs, -tau), 0.f);
            pe[c] = c < lim ? pow_e(mm, ei, e) : 0.f;
          }
          chunk_step(k, pe);
        }
      }
      ptx::tmem_wait_st();
#pragma unroll
      for (int o = 1; o < G; o <<= 1) slog += __shfl_xor_sync(0xffffffffu, slog, o);
      // counts and sums of log w of the other blocks: total for mu, lower ranks for the list position
      ok = exchange((float)nsel, slog);
      // (counts are small integers: exact in fp32)
      const int nsel_all = (int)x_sum_a;
      int base = (int)x_below_a;
      const float slog_all = x_sum_b;
      if (row_valid && hh == 0 && my_rank == 0) {
        for (int j = (n_cand + 31) / 32; j < dm.W; ++j) mrow[j] = ((c_own >> 5) == j) ? (1u << (c_own & 31)) : 0u;
        a.count[row_id] = nsel_all;
      }
      const float mu = nsel_all > 0 ? slog_all / (float)nsel_all : 0.f;
      for (int k = in_regs ? 0 : k_lo; k < (in_regs ? n_chunks : k_hi) && ok; ++k) {
        uint32_t lwv[OWN];
        ptx::tmem_ld_n<OWN>(lwv, lane_addr + k * 32);
        ptx::tmem_wait_ld();
        uint32_t bits = 0;
#pragma unroll
        for (int q = 0; q < OWN; ++q)
          if (lwv[q] != 0x7f800000u) bits |= 1u << (own0 + q);
#pragma unroll
        for (int o = 1; o < G; o <<= 1) bits |= __shfl_xor_sync(0xffffffffu, bits, o);
        if (row_valid) {
#pragma unroll
          for (int q = 0; q < OWN; ++q) {
            if (lwv[q] != 0x7f800000u) {
              const int c = own0 + q;
              const long long pos = loff + base + __popc(bits & ((1u << c) - 1u));
              a.blk_bias[pos] = (__uint_as_float(lwv[q]) - mu) * dm.inv_sigma;
              if (a.blk_idx) a.blk_idx[pos] = c_lo + k * 32 + c;
            }
          }
        }
        base += __popc(bits);
      }
    }
    };
    if (e_int == 2) solve(std::integral_constant<int, 2>{}); else solve(std::integral_constant<int, -1>{});
    ptx::tc_fence_before();
  }

  __syncthreads();
  if (warp == W_MMA) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, a.tmem_cols);
  }
  if (tid == 0 && misc->abort_flag) report_error(a.sb, DASH_ERR_TIMEOUT, 201);
  if (CS > 1) ptx::cluster_sync_all();     // nobody leaves while a peer may still write into its shared memory
}

}  // namespace

// Tokens [0, select_sm100_token_limit) can be routed by the tensor-core kernel (0: not applicable).  A block
// holds 512 candidates per row in tensor memory; clusters of 2 or 4 blocks extend that to 1024 / 2048.
int select_sm100_token_limit(const Dims& dm) {
  if (dm.decode || !dm.causal || dm.dtype != DASH_BF16 || (dm.d != 64 && dm.d != 128) || dm.T_s < 1) return 0;
  if (dm.g_q < 2) return 0;
  if (tensor_map_encoder() == nullptr) return 0;
  const long long lim = (long long)(4 * CLUSTER_COLS + 1) * dm.B;   // own chunk index <= 2048
  return (int)(lim < dm.seq_q ? lim : dm.seq_q);
}

size_t select_sm100_scratch_bytes(const Dims& dm) {
  return (size_t)3 * dm.batch * dm.h_kv * (size_t)(dm.T_s > 0 ? dm.T_s : 1) * dm.d * sizeof(__nv_bfloat16);
}

template <int NST, int G, int CS, int HD, bool SHORT = false>
static cudaError_t launch_band(const CUtensorMap& tq, const CUtensorMap& tkb, const SelectTcArgs& a, long long clusters,
                               cudaStream_t st) {
  auto kern = select_sm100_kernel<NST, G, CS, HD, SHORT>;
  static std::atomic<unsigned long long> configured{0};
  if (cudaError_t e = allow_dynamic_smem(kern, SmemPlan<NST>::TOTAL, configured); e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(clusters * CS));
  cfg.blockDim = dim3(sel_threads(NST));
  cfg.dynamicSmemBytes = SmemPlan<NST>::TOTAL;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see launch_chained
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tq, tkb, a);
  count_launch();
  return e;
}

template <int NST, int CS>
static cudaError_t launch_band_g(const Dims& dm, const CUtensorMap& tq, const CUtensorMap& tkb, const SelectTcArgs& a,
                                 long long clusters, cudaStream_t st) {
  if (a.TQ * dm.g_q < 128) {      // short tiles: only g_q = 2 (chunks of 16 or 32) and g_q = 4 (chunks of 16)
    if (dm.d == 64) {
      if (dm.g_q == 2) return launch_band<NST, 2, CS, 64, true>(tq, tkb, a, clusters, st);
      if (dm.g_q == 4) return launch_band<NST, 4, CS, 64, true>(tq, tkb, a, clusters, st);
    } else {
      if (dm.g_q == 2) return launch_band<NST, 2, CS, 128, true>(tq, tkb, a, clusters, st);
      if (dm.g_q == 4) return launch_band<NST, 4, CS, 128, true>(tq, tkb, a, clusters, st);
    }
    return cudaErrorInvalidValue;
  }
  if (dm.d == 64) {
    switch (dm.g_q) {
      case 2: return launch_band<NST, 2, CS, 64>(tq, tkb, a, clusters, st);
      case 4: return launch_band<NST, 4, CS, 64>(tq, tkb, a, clusters, st);
      case 8: return launch_band<NST, 8, CS, 64>(tq, tkb, a, clusters, st);
      case 16: return launch_band<NST, 16, CS, 64>(tq, tkb, a, clusters, st);
      default: return cudaErrorInvalidValue;
    }
  }
  switch (dm.g_q) {
    case 2: return launch_band<NST, 2, CS, 128>(tq, tkb, a, clusters, st);
    case 4: return launch_band<NST, 4, CS, 128>(tq, tkb, a, clusters, st);
    case 8: return launch_band<NST, 8, CS, 128>(tq, tkb, a, clusters, st);
    case 16: return launch_band<NST, 16, CS, 128>(tq, tkb, a, clusters, st);
    default: return cudaErrorInvalidValue;
  }
}

// Local window: the chunks [c_own - L, c_own) of every row are attended with bias 0 without being scored.  The
// routing kernel above leaves them out; this one (launched behind it only when L > 0) sets their mask bits,
// appends them to the row's list behind the routed chunks and adds them to the count.  One thread per row.
__global__ void __launch_bounds__(256)
window_rows_kernel(Dims dm, int token_limit, uint32_t* __restrict__ mask, int* __restrict__ count,
                   int* __restrict__ blk_idx, float* __restrict__ blk_bias) {
  chain_wait();
  chain_release();
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long total = (long long)dm.batch * dm.h_kv * token_limit;
  if (idx >= total) return;
  const int i = (int)(idx % token_limit);
  const long long grp = idx / token_limit;
  const int n_vis = min(i / dm.B, dm.T_s);
  const int n_cand = max(n_vis - dm.local_blocks, 0);
  if (n_vis == n_cand) return;
  const long long row_id = grp * dm.seq_q + i;
  uint32_t* mrow = mask + row_id * dm.W;
  const int routed = count[row_id];
  const long long loff = grp * dm.list_rows + list_row_offset(dm, i) + routed;
  for (int c = n_cand; c < n_vis; ++c) {
    mrow[c >> 5] |= 1u << (c & 31);
    blk_bias[loff + (c - n_cand)] = 0.f;
    if (blk_idx) blk_idx[loff + (c - n_cand)] = c;
  }
  count[row_id] = routed + (n_vis - n_cand);
}

cudaError_t launch_select_sm100(const Dims& dm, int token_limit, const void* Q, const float* Kbar, void* planes,
                                uint32_t* mask, int* count, int* blk_idx, float* blk_bias, float* tau,
                                StatusBlock* sb, cudaStream_t st, bool planes_ready) {
  const long long plane_rows = (long long)dm.batch * dm.h_kv * dm.T_s;
  const long long n = plane_rows * dm.d;
  cudaError_t e = cudaSuccess;
  if (!planes_ready) {       // the summaries came from the caller: split them here
    e = launch_chained(kbar_split_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, Kbar,
                       (__nv_bfloat16*)planes, n);
    count_launch();
    if (e != cudaSuccess) return e;
  }

  SelectTcArgs a;
  a.dm = dm;
  a.TQ = 128 / dm.g_q < dm.B ? 128 / dm.g_q : dm.B;     // a tile stays inside one chunk
  a.plane_rows = plane_rows;
  a.mask = mask; a.count = count; a.blk_idx = blk_idx; a.blk_bias = blk_bias; a.tau = tau; a.sb = sb;

  CUtensorMap tq, tkb;
  {
    cuuint64_t dims[4] = {(cuuint64_t)dm.d, (cuuint64_t)dm.h_q, (cuuint64_t)dm.seq_q, (cuuint64_t)dm.batch};
    auto sb2 = [](long long el) { return (cuuint64_t)((el > 0 ? el : 8) * 2); };
    cuuint64_t strides[3] = {sb2(dm.qs[2]), sb2(dm.qs[1]), sb2(dm.qs[0])};
    cuuint32_t box[4] = {64u, (cuuint32_t)dm.g_q, (cuuint32_t)a.TQ, 1u};
    if (!encode_bf16_sw128_4d(&tq, Q, dims, strides, box)) return cudaErrorInvalidValue;
  }
  {
    const cuuint64_t hd = (cuuint64_t)dm.d;
    cuuint64_t dims[4] = {hd, (cuuint64_t)(3 * plane_rows), 1, 1};
    cuuint64_t strides[3] = {hd * 2, (cuuint64_t)(3 * plane_rows) * hd * 2, (cuuint64_t)(3 * plane_rows) * hd * 2};
    cuuint32_t box[4] = {64u, (cuuint32_t)SC, 1u, 1u};
    if (!encode_bf16_sw128_4d(&tkb, planes, dims, strides, box)) return cudaErrorInvalidValue;
  }
  // Bands of tiles by candidate count: <= 512 one block per tile, <= 1024 clusters of 2, <= 2048 clusters of 4.
  // Tiles are TQ tokens; a tile's candidate count is its own chunk index i0 / B.
  const int groups = dm.batch * dm.h_kv;
  const int total_tiles = (token_limit + a.TQ - 1) / a.TQ;
  auto tiles_up_to = [&](long long max_cand) -> int {      // tiles whose own chunk index is <= max_cand
    const long long tokens = (max_cand + 1) * dm.B;
    const long long t = (tokens + a.TQ - 1) / a.TQ;
    return (int)(t < total_tiles ? t : total_tiles);
  };
  const int t1 = tiles_up_to(CLUSTER_COLS), t2 = tiles_up_to(2 * CLUSTER_COLS), t3 = total_tiles;
  // widest bands first: they are the long-running ones
  if (t3 > t2) {
    a.tile_base = t2; a.n_tiles = t3 - t2; a.tmem_cols = 512;
    if ((e = launch_band_g<3, 4>(dm, tq, tkb, a, (long long)a.n_tiles * groups, st)) != cudaSuccess) return e;
  }
  if (t2 > t1) {
    a.tile_base = t1; a.n_tiles = t2 - t1; a.tmem_cols = 512;
    if ((e = launch_band_g<3, 2>(dm, tq, tkb, a, (long long)a.n_tiles * groups, st)) != cudaSuccess) return e;
  }
  // one block per tile: rows of 257 .. 512 candidates take the whole tensor memory of an SM (one block per SM, three
  // solver threads per row); shorter ones leave room for two blocks per SM with the row in one thread
  const int t0 = tiles_up_to(256);
  if (t1 > t0) {
    a.tile_base = t0; a.n_tiles = t1 - t0; a.tmem_cols = 512;
    if ((e = launch_band_g<3, 1>(dm, tq, tkb, a, (long long)a.n_tiles * groups, st)) != cudaSuccess) return e;
  }
  {
    a.tile_base = 0; a.n_tiles = t0;
    const int max_cand = min(dm.T_s, (int)(((long long)t0 * a.TQ - 1) / dm.B));
    uint32_t cols = 32;
    while ((int)cols < ((max_cand + SC - 1) / SC) * SC) cols <<= 1;
    a.tmem_cols = cols;
    e = launch_band_g<1, 1>(dm, tq, tkb, a, (long long)a.n_tiles * groups, st);
  }
  if (e == cudaSuccess && dm.local_blocks > 0) {
    const long long rows = (long long)groups * token_limit;
    e = launch_chained(window_rows_kernel, dim3((unsigned)((rows + 255) / 256)), dim3(256), 0, st, dm, token_limit,
                       mask, count, blk_idx, blk_bias);
    count_launch();
  }
  return e;
}

}  // namespace dash
