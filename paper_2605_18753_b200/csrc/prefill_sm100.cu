// Stage 2, prefill, tensor-core path for sm_100a (Eq. 7 in the form of Proposition 1; Algorithm 3).
//
// Tile: one (batch, KV head) and TQ = min(128/g_q, chunk size) consecutive query tokens; the rows of the MMA tile
// are (token, head-of-group) pairs, token-major (with chunks shorter than 128/g_q tokens the tile holds fewer than
// 128 live rows; the rest are zero queries whose results are dropped).  A tile never straddles a chunk, so its rows share the own
// chunk; it takes the own chunk first (its tiles can be fetched before the mask has been read), then walks
// the UNION of its rows' routed chunks in ascending order, 64 KV tokens per step.  A row that did not route
// a chunk gets bias -inf for that step (probability exactly 0), so every row still attends to its own
// selection only.
//
// Warp roles (256 threads = two warpgroups, two blocks per SM so one block's softmax overlaps the other's MMAs; after
// set-up the second warpgroup hands most of its registers to the first with setmaxnreg):
//   warps 0-3  softmax: S (TMEM) -> registers, logit = S/sqrt(d) + bias, causal mask inside the own chunk,
//              online softmax with a lazily moved row maximum, P (bf16) -> TMEM over the S columns, rescale of
//              the O accumulator in TMEM when the maximum moved, final O / l -> global.
//   warp 4     K producer: TMA loads of Q and of the K tiles (128-byte swizzle, no multicast); OR of the tile's
//              mask words = union list.
//   warp 6     V producer: walks the same union list; TMA loads of the V tiles and the per-token bias of each
//              step (a row's list entry for a chunk = its routed bits below the chunk + the totals of the earlier mask
//              words: read by direct index, a whole step's loads issued together before the wait for the stage).
//   warp 5     MMA issuer: S_{j+1} = Q K_{j+1}^T (M128 N64 K128) into one of two TMEM buffers, then O += P_j V_j
//              (M128 N128 K64, P from TMEM); one tcgen05.commit per product, to the mbarrier that the softmax
//              warps and the producer of the stage both listen to; owns the TMEM allocation.
//   warp 7     idle (it completes the second warpgroup: registers are re-divided per whole warpgroup).
// Every wait is bounded; a wait that runs out raises DASH_ERR_TIMEOUT in the status word and every role
// leaves its loop, frees TMEM and returns.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace dash {

namespace {

constexpr int NKV = 64;           // KV tokens per step
constexpr int KST = 2, VST = 2;   // ring depths: stage = step parity, like the S/P buffers, so that the two
                                  // MMA completion barriers of a step also release its K and V stages
constexpr int PF_THREADS = 256;   // 4 softmax warps, K producer, MMA issuer, V/bias producer and an idle warp: two whole
                                  // warpgroups, because a warpgroup changes its register budget only when all four of
                                  // its warps ask (a block of seven warps waits for the eighth for ever)
// Registers per thread after the re-division (two blocks per SM start with 128 each): 128 * (200 - 128) taken by the
// softmax warpgroup = 128 * (128 - 56) given up by the other one; the block's own pool is all that it can draw from.
constexpr int PF_REGS_SERVICE = 56, PF_REGS_SOFTMAX = 200;
static_assert(PF_THREADS == 256 && 128 * (PF_REGS_SOFTMAX - 128) <= 128 * (128 - PF_REGS_SERVICE),
              "the softmax warpgroup can only take what the service warpgroup released: a larger request never completes");
constexpr uint32_t TMEM_COLS = 256;  // S0 [0,64), S1 [64,128), O [128,256)
constexpr float RESCALE_LOG2 = 8.f;  // the running maximum is moved only when it grew by more than this

constexpr int MAX_TQ = 64;
// S_FULL[j&1]: QK of step j complete (S readable; K stage j&1 reusable).  PV_DONE[j&1]: PV of step j complete (O stable;
// S/P buffer and V stage j&1 reusable).  Every tcgen05.commit and every barrier test costs the issuing thread as
// much as an MMA, so each product signals exactly one barrier and the producers listen to the same ones.
enum Bar { Q_FULL = 0, META, S_FULL = 2, PV_DONE = 4, P_FULL = 6, V_FULL = 8, K_FULL = 10, N_BARS = 12 };
static_assert(KST == 2 && VST == 2, "stage = step parity");
// CPS = chunks per 64-token step: 1 for chunks of 64 or 128 tokens, 2 / 4 for chunks of 32 / 16 (a step then
// packs that many chunks of the union list, each with its own per-token bias).
template <int CPS>
struct MiscT {
  unsigned long long bar[N_BARS];
  uint32_t tmem_base;
  int n_steps;
  int abort_flag;
  int kvbase[VST][CPS];
  float bias[VST][CPS][MAX_TQ];
};
// Shared-memory layout for head_dim HD (64 or 128): tiles are K-major regions of 64 elements (128 bytes, the
// swizzle span) per row, one region per 64 of head_dim.
template <int HD, int CPS>
struct PfLayout {
  static constexpr uint32_t Q_BYTES = 128 * HD * 2;           // HD = 128: 32 KiB, two 128x64 regions
  static constexpr uint32_t KV_TILE_BYTES = NKV * HD * 2;     // HD = 128: 16 KiB, two 64x64 regions
  static constexpr uint32_t OFF_Q = 0;
  static constexpr uint32_t OFF_K = OFF_Q + Q_BYTES;
  static constexpr uint32_t OFF_V = OFF_K + KST * KV_TILE_BYTES;
  static constexpr uint32_t OFF_MISC = OFF_V + VST * KV_TILE_BYTES;
  static constexpr uint32_t SMEM = OFF_MISC + sizeof(MiscT<CPS>);
  static_assert(SMEM <= 115712, "two blocks per SM need <= 113 KiB each");
};


// max of three in one instruction
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

struct PrefillArgs {
  Dims dm;
  int TQ;            // tokens per tile
  int n_tiles;       // tiles per (batch, KV head)
  int early_loads;   // 1: Q, K, V are not written by the kernel before this one on the stream (their first loads may precede chain_wait)
  int inject;        // test hook: 1 = the K producer never loads the own chunk's keys (the waits for them run out)
  long long wait_limit;   // cycles a bounded wait may spin
  const uint32_t* mask;
  const float* blk_bias;
  __nv_bfloat16* O;          // may be null when only the row statistics are wanted
  // Row statistics for the backward pass, [batch][KV head][tile][row of the tile (128)] (null: not wanted): the
  // log-sum-exp of the row's logits in the log2 domain, and delta = <O_row, dO_row> (dO: strides of O), both from the
  // fp32 accumulator.
  float* lse2;
  float* delta;
  const __nv_bfloat16* dO;
  StatusBlock* sb;
};

// SHORT: the tile has fewer than 128 live rows (chunks shorter than 128 / g_q tokens); full tiles compile without
// any of the padding-row handling.
// STATS: the kernel also leaves the row statistics the backward pass starts from (a.lse2, a.delta).  delta = <O, dO> feeds
// the gradient of the routing, which amplifies its error, so in this mode P enters the P V product as two bf16 terms
// (P = hi + lo, the remainder in the second half of the step's S columns): O, and with it delta, is then accurate to
// fp32 class instead of bf16 class.
template <int HD, int CPS, bool SHORT, bool STATS = false>
__global__ void __launch_bounds__(PF_THREADS, 2)
attend_prefill_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                            const __grid_constant__ CUtensorMap tmV, PrefillArgs a) {
  using LY = PfLayout<HD, CPS>;
  using Misc = MiscT<CPS>;
  constexpr uint32_t Q_BYTES = LY::Q_BYTES, KV_TILE_BYTES = LY::KV_TILE_BYTES, OFF_Q = LY::OFF_Q, OFF_K = LY::OFF_K,
                     OFF_V = LY::OFF_V, OFF_MISC = LY::OFF_MISC;
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
  const int sub_per_blk = dm.B / NKV;                 // 64-token steps per chunk (1 or 2)
  const int own_steps = (i0 % dm.B) / NKV + 1;        // steps of the own chunk the tile can see

  if (tid == 0) {
    if ((sbase & 1023u) != 0u) {
      report_error(a.sb, DASH_ERR_CUDA, 100);
      misc->abort_flag = 1;
    } else {
      misc->abort_flag = 0;
    }
    ptx::mbar_init(bar(Q_FULL), 1);
    ptx::mbar_init(bar(META), 1);
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(bar(S_FULL + s), 1);
      ptx::mbar_init(bar(PV_DONE + s), 1);
      ptx::mbar_init(bar(K_FULL + s), 1);
      ptx::mbar_init(bar(V_FULL + s), 1);
    }
    // two P_FULL barriers (step parity): the softmax warps may finish step j+1 before the MMA thread has
    // looked at step j, and a single barrier's phase bit cannot tell j from j+2
    ptx::mbar_init(bar(P_FULL), 128);
    ptx::mbar_init(bar(P_FULL + 1), 128);
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
  // Rows of the Q tile beyond the tile's TQ * g_q live rows (chunks shorter than 128 / g_q tokens) are never written by
  // the TMA box: they are zeroed once, so that their scores are finite; their probabilities are forced to 0 below.
  if constexpr (SHORT) {
    const int first = TQ * g_q * 8;                 // 16-byte pieces before the first dead row (a row is 128 bytes)
    for (int regn = 0; regn < HD / 64; ++regn)
      for (int k = first + tid; k < 128 * 8; k += PF_THREADS)
        *reinterpret_cast<uint4*>(smem + OFF_Q + regn * (Q_BYTES / (HD / 64)) + k * 16) = make_uint4(0u, 0u, 0u, 0u);
    ptx::fence_proxy_async_smem();
  }
  // A step's K or V tile for chunks smaller than the step: CPS boxes of NKV / CPS tokens, one per packed chunk.
  [[maybe_unused]] auto load_packed = [&](const CUtensorMap* tm, uint32_t dst, uint32_t barrier, const int* kvs) {
    ptx::mbar_arrive_expect_tx(barrier, KV_TILE_BYTES);
#pragma unroll
    for (int s = 0; s < CPS; ++s) {
      const uint32_t d = dst + s * (NKV / CPS) * 128;
      ptx::tma_load_4d(d, tm, barrier, 0, r, kvs[s], b);
      if constexpr (HD == 128) ptx::tma_load_4d(d + KV_TILE_BYTES / 2, tm, barrier, 64, r, kvs[s], b);
    }
  };
  // Q and the own chunk's K / V tiles: they need nothing from the routing kernels (and go first anyway).
  auto own_loads = [&](bool do_k, bool do_v) {
    const int TR = SHORT ? 128 / g_q : TQ;
    if (lane == 0 && do_k) {
      ptx::prefetch_tensormap(&tmQ);
      ptx::prefetch_tensormap(&tmK);
      ptx::prefetch_tensormap(&tmV);
      ptx::mbar_arrive_expect_tx(bar(Q_FULL), SHORT ? (uint32_t)(TQ * g_q * HD * 2) : Q_BYTES);   // the box holds the live rows
      ptx::tma_load_4d(sbase + OFF_Q, &tmQ, bar(Q_FULL), 0, r * g_q, i0, b);
      if constexpr (HD == 128) ptx::tma_load_4d(sbase + OFF_Q + Q_BYTES / 2, &tmQ, bar(Q_FULL), 64, r * g_q, i0, b);
    }
    // The own chunk goes first: its tiles need nothing from the mask, so they are in flight (and the first
    // S = Q K^T can run) while the union of the routed chunks is still being formed.  Stages 0/1 are free.
    for (int sub = 0; sub < own_steps; ++sub) {
      const int kv0 = c_own * dm.B + sub * NKV;
      if constexpr (CPS > 1) {
        // the own chunk fills the first slot of step 0; the other slots repeat it with bias -inf (probability 0)
        int kvs[CPS];
#pragma unroll
        for (int s = 0; s < CPS; ++s) kvs[s] = kv0;
        if (do_k) {
          if (lane == 0 && !a.inject) load_packed(&tmK, sbase + OFF_K, bar(K_FULL), kvs);
        } else {
          for (int t = lane; t < TR; t += 32) {
            misc->bias[0][0][t] = t < TQ ? 0.f : -INFINITY;     // token slots beyond TQ: padding rows of a short tile
#pragma unroll
            for (int s = 1; s < CPS; ++s) misc->bias[0][s][t] = -INFINITY;
          }
          if (lane < CPS) misc->kvbase[0][lane] = kv0;
          __syncwarp();
          if (lane == 0) load_packed(&tmV, sbase + OFF_V, bar(V_FULL), kvs);
        }
        continue;
      }
      if (do_k) {
        if (lane == 0 && !a.inject) {
          const uint32_t dst = sbase + OFF_K + sub * KV_TILE_BYTES;
          ptx::mbar_arrive_expect_tx(bar(K_FULL + sub), KV_TILE_BYTES);
          ptx::tma_load_4d(dst, &tmK, bar(K_FULL + sub), 0, r, kv0, b);
          if constexpr (HD == 128) ptx::tma_load_4d(dst + KV_TILE_BYTES / 2, &tmK, bar(K_FULL + sub), 64, r, kv0, b);
        }
      } else {
        for (int t = lane; t < TR; t += 32) misc->bias[sub][0][t] = t < TQ ? 0.f : -INFINITY;   // beyond TQ: padding rows
        if (lane == 0) misc->kvbase[sub][0] = kv0;
        __syncwarp();
        if (lane == 0) {
          const uint32_t dst = sbase + OFF_V + sub * KV_TILE_BYTES;
          ptx::mbar_arrive_expect_tx(bar(V_FULL + sub), KV_TILE_BYTES);
          ptx::tma_load_4d(dst, &tmV, bar(V_FULL + sub), 0, r, kv0, b);
          if constexpr (HD == 128) ptx::tma_load_4d(dst + KV_TILE_BYTES / 2, &tmV, bar(V_FULL + sub), 64, r, kv0, b);
        }
      }
    }
  };
  // Q, K and V are inputs of the whole chain, not outputs of the kernel before this one: when the caller vouches for
  // that, their first tiles are under way while that kernel still drains
  if (a.early_loads && (warp == 4 || warp == 6)) own_loads(warp == 4, warp == 6);
  // barriers and tensor memory are set up; from here on the kernel reads what the routing kernels wrote
  chain_wait();
  chain_release();
  // a workspace whose status word already holds an error makes every role leave at its first wait: after one
  // block's wait has run out, the rest of the grid retires in microseconds instead of a wait limit each
  if (a.sb && *reinterpret_cast<volatile int*>(&a.sb->status) != 0) *abort_flag = 1;
  __syncthreads();

  if (warp >= 4) {
  // the register file of the block is re-divided between its two warpgroups: this one gives up what the softmax
  // warpgroup takes (each side opens with its own instruction, so the allocator knows the budget of each)
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PF_REGS_SERVICE));
  if (warp == 4 || warp == 6) {
    // =========================== producers ===========================
    // Two warps walk the same union list: warp 4 feeds the K ring (and loads Q), warp 6 feeds the V ring and
    // the per-token bias of each step.  Split like this, a full V ring never holds back the next K tile.
    const bool do_k = (warp == 4), do_v = (warp == 6);
    const int TR = SHORT ? 128 / g_q : TQ;   // token slots of the 128 tile rows; slots TQ .. TR-1 are padding (bias -inf)
    if (!a.early_loads) own_loads(do_k, do_v);
    // union of the tile's mask words (lane t owns tokens t, t+32)
    const int n_words = (c_own >> 5) + 1;
    const long long row0 = ((long long)b * dm.h_kv + r) * dm.seq_q;
    const uint32_t own_word_keep = (c_own & 31) == 31 ? 0xffffffffu : ((2u << (c_own & 31)) - 1u);
    // four mask words per sweep: a lane's eight loads are in flight together (one L2 round trip per four words
    // instead of one per word; the step count below is what the MMA thread waits for before its second product)
    int total = 0;
    for (int w0 = 0; w0 < n_words; w0 += 4) {
      uint32_t uu[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int t = lane + 32 * q;
        if (t < TQ && i0 + t < dm.seq_q) {
          const uint32_t* mp = a.mask + (row0 + i0 + t) * dm.W + w0;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if (w0 + k < n_words) uu[k] |= mp[k];
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (w0 + k < n_words) {
          uint32_t u = __reduce_or_sync(0xffffffffu, uu[k]);
          if (w0 + k == n_words - 1) u = (u & own_word_keep) | (1u << (c_own & 31));  // own chunk: always, and last
          total += __popc(u);
        }
      }
    }
    // the own chunk is always in the union (its bit is set in every row); it contributes own_steps steps
    const int n_steps = CPS > 1 ? (total - 1 + CPS - 1) / CPS + own_steps : (total - 1) * sub_per_blk + own_steps;
    if (lane == 0 && do_k) {
      misc->n_steps = n_steps;
      ptx::mbar_arrive(bar(META));
    }
    // start of the compact bias lists of this lane's tokens (lane t owns tokens t and t+32)
    long long loff[2];
    for (int q = 0; q < 2; ++q) {
      const int t = lane + 32 * q;
      const int i = min(i0 + t, dm.seq_q - 1);
      loff[q] = ((long long)b * dm.h_kv + r) * dm.list_rows + list_row_offset(dm, i);
    }
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
    // The walk pops the chunks of the union in ascending order; mask words are read one word ahead.
    int w = 0;
    uint32_t rw[2], rw_n[2] = {0u, 0u};
    load_rows(0, rw);
    uint32_t u = union_of(0, rw);
    if (n_words > 1) load_rows(1, rw_n);
    int j = own_steps;                 // the own chunk's steps are already under way
    bool ok = true;
    // last step loaded into each stage (-1: none): what a block that gives up has to let land before it retires
    int last_j[2] = {-1, -1};
    for (int sub = 0; sub < (CPS > 1 ? 1 : own_steps); ++sub) last_j[sub] = (do_k && a.inject) ? -1 : sub;
    {
      // A step takes the next CPS chunks of the union (CPS > 1: chunks of 32 / 16 tokens packed into the 64-token
      // step; a short last step repeats its last chunk with bias -inf).  A row's bias for a chunk is read straight
      // from its list: the entry number is the count of the row's routed bits below the chunk (previous words'
      // totals kept in `seen`), so the loads of a whole step are issued together, before the wait for the stage,
      // and nothing walks the lists entry by entry.
      int seen[2] = {0, 0};
      auto routed_bits = [&](uint32_t word) -> uint32_t {    // a row's routed chunks in word w: the own chunk and later ones cleared
        return w == n_words - 1 ? word & own_word_keep & ~(1u << (c_own & 31)) : word;
      };
      bool walking = true;
      while (walking && ok) {
        int cs[CPS];
        float bvs[CPS][2];
        int m = 0;
        while (m < CPS) {
          while (u == 0u && walking) {
            seen[0] += __popc(routed_bits(rw[0]));
            seen[1] += __popc(routed_bits(rw[1]));
            if (++w >= n_words) { walking = false; break; }
            rw[0] = rw_n[0]; rw[1] = rw_n[1];
            u = union_of(w, rw);
            if (w + 1 < n_words) load_rows(w + 1, rw_n);
          }
          if (!walking) break;
          const int bit = __ffs(u) - 1;
          u &= u - 1;
          const int c = w * 32 + bit;
          if (c == c_own) { walking = false; break; }        // last of the walk, done first
          cs[m] = c;
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const uint32_t rb = routed_bits(rw[q]);
            const bool member = do_v && ((rb >> bit) & 1u);
            const int e = seen[q] + __popc(rb & ((1u << bit) - 1u));
            bvs[m][q] = member ? __ldg(a.blk_bias + loff[q] + e) : -INFINITY;
          }
          ++m;
        }
        if (m == 0) break;
#pragma unroll
        for (int s = 1; s < CPS; ++s)
          if (s >= m) { cs[s] = cs[m - 1]; bvs[s][0] = bvs[s][1] = -INFINITY; }
        // chunks of 128 tokens take two 64-token steps with the same bias
        for (int sub = 0; sub < (CPS > 1 ? 1 : sub_per_blk) && ok; ++sub, ++j) {
          int kvs[CPS];
#pragma unroll
          for (int s = 0; s < CPS; ++s) kvs[s] = cs[s] * dm.B + sub * NKV;
          const int st = j & 1, prev_ph = ((j >> 1) - 1) & 1;   // stage, and the phase of step j-2 on the completion barriers
          if (do_k) {
            if (j >= 2) ok = wait_on(bar(S_FULL + st), prev_ph);     // QK of step j-2 has read the stage
            if (!ok) break;
            if (lane == 0) load_packed(&tmK, sbase + OFF_K + st * KV_TILE_BYTES, bar(K_FULL + st), kvs);
            last_j[st] = j;
          } else {
            if (j >= 2) ok = wait_on(bar(PV_DONE + st), prev_ph);    // PV of step j-2 has read the stage
            if (!ok) break;
#pragma unroll
            for (int s = 0; s < CPS; ++s)
              for (int q = 0; q < 2; ++q) {
                const int t = lane + 32 * q;
                if (t < TR) misc->bias[st][s][t] = t < TQ ? bvs[s][q] : -INFINITY;
              }
#pragma unroll
            for (int s = 0; s < CPS; ++s)
              if (lane == s) misc->kvbase[st][s] = kvs[s];
            __syncwarp();
            if (lane == 0) load_packed(&tmV, sbase + OFF_V + st * KV_TILE_BYTES, bar(V_FULL + st), kvs);
            last_j[st] = j;
          }
        }
      }
    }
    if (!ok && lane == 0) {
      // a wait ran out: let the copies already issued land (bounded) before the block retires
      for (int s = 0; s < 2; ++s) {
        if (last_j[s] < 0) continue;
        const uint32_t full = bar((do_k ? K_FULL : V_FULL) + s), parity = (uint32_t)(last_j[s] >> 1) & 1u;
        for (int k = 0; k < 200000 && !ptx::mbar_try_wait(full, parity); ++k) {}
      }
      if (do_k)
        for (int k = 0; k < 200000 && !ptx::mbar_try_wait(bar(Q_FULL), 0); ++k) {}
    }
  } else if (warp == 5) {
    // =========================== MMA issuer ===========================
    // Per step: S_{j+1} = Q K_{j+1}^T (needs only its K tile), then O += P_j V_j.  V_FULL is not tested here: the
    // softmax threads wait for it (the step's bias arrives with it) before they arrive on P_FULL.
    if (lane == 0) {
      bool ok = wait_on(bar(Q_FULL), 0);
      constexpr uint32_t IDESC_QK = ptx::idesc_bf16_f32(128, NKV, false, false);
      constexpr uint32_t IDESC_PV = ptx::idesc_bf16_f32(128, HD, false, true);
      // Descriptors differ only in the 14-bit start-address field (16-byte units, no carry into the next
      // field): build them once, then a single add per MMA keeps the issuing thread's instruction stream short.
      const uint64_t qd0 = ptx::smem_desc_sw128(sbase + OFF_Q, 16, 1024);
      const uint64_t kd0 = ptx::smem_desc_sw128(sbase + OFF_K, 16, 1024);
      const uint64_t vd0 = ptx::smem_desc_sw128(sbase + OFF_V, KV_TILE_BYTES / 2, 1024);
      auto issue_qk = [&](int j) -> bool {
        const int buf = j & 1;
        if (!wait_on(bar(K_FULL + buf), (j >> 1) & 1)) return false;
        // the S/P buffer is recycled in MMA issue order (PV of step j-2 precedes this QK)
        ptx::tc_fence_after();
        const uint64_t kd = kd0 + (uint64_t)((buf * KV_TILE_BYTES) >> 4);
        const uint32_t d_tmem = tmem + buf * NKV;
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          // 16 bf16 = 32 bytes inside the 128-byte swizzle row; the second 64 columns live in the next region
          const uint64_t ad = qd0 + (uint64_t)(((k >> 2) * (Q_BYTES / 2) + (k & 3) * 32) >> 4);
          const uint64_t bd = kd + (uint64_t)(((k >> 2) * (KV_TILE_BYTES / 2) + (k & 3) * 32) >> 4);
          ptx::mma_bf16_ss(d_tmem, ad, bd, IDESC_QK, k > 0 ? 1u : 0u);
        }
        ptx::mma_commit(bar(S_FULL + buf));
        return true;
      };
      if (ok) ok = issue_qk(0);          // the own chunk: there is always a step 0, whatever the union holds
      ok = ok && wait_on(bar(META), 0);
      const int n_steps = ok ? misc->n_steps : 0;
      for (int j = 0; j < n_steps && ok; ++j) {
        if (j + 1 < n_steps) ok = issue_qk(j + 1);
        if (!ok) break;
        const int buf = j & 1;
        ok = wait_on(bar(P_FULL + buf), (j >> 1) & 1);
        if (!ok) break;
        ptx::tc_fence_after();
        // V is [kv token][d]: MN-major B operand; 64-wide d blocks are KV_TILE_BYTES/2 apart; 16 tokens = 2048 bytes
        const uint64_t vd = vd0 + (uint64_t)((buf * KV_TILE_BYTES) >> 4);
        const uint32_t p_tmem = tmem + buf * NKV;
#pragma unroll
        for (int k = 0; k < NKV / 16; ++k) {
          const uint64_t bd = vd + (uint64_t)((k * 16 * 128) >> 4);
          // A = P from tensor memory: 16 bf16 per K step = 8 packed columns
          ptx::mma_bf16_ts(tmem + 2 * NKV, p_tmem + k * 8, bd, IDESC_PV, (j > 0 || k > 0) ? 1u : 0u);
        }
        if constexpr (STATS) {
#pragma unroll
          for (int k = 0; k < NKV / 16; ++k) {
            const uint64_t bd = vd + (uint64_t)((k * 16 * 128) >> 4);
            ptx::mma_bf16_ts(tmem + 2 * NKV, p_tmem + 32 + k * 8, bd, IDESC_PV, 1u);      // the remainders
          }
        }
        ptx::mma_commit(bar(PV_DONE + buf));
      }
    }
    __syncwarp();
  }
  } else {
    // =========================== softmax / epilogue ===========================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(PF_REGS_SOFTMAX));
    const int m = tid;                       // tile row = TMEM lane
    const int t = m / g_q, hh = m % g_q;     // token in tile, head in group
    const int i_row = i0 + t;
    const bool row_live = t < TQ;            // false for the padding rows of a tile shorter than 128 rows
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    const float c1 = dm.sm_scale * 1.4426950408889634f;
    bool ok = true;
    int n_steps = 0x7fffffff;                // known from step 1 on; step 0 (the own chunk) always exists
    float m_used = -INFINITY, l = 0.f;

    for (int j = 0; ok; ++j) {
      if (j == 1) {
        ok = wait_on(bar(META), 0);
        if (!ok) break;
        n_steps = misc->n_steps;
      }
      if (j >= n_steps) break;
      const int buf = j & 1;
      // bias / kvbase of the step visible; the MMA thread relies on this wait for the V tile as well
      ok = wait_on(bar(V_FULL + buf), (j >> 1) & 1);
      if (!ok) break;
      float b2s[CPS];                                // per packed chunk: bias in the log2 domain (-inf: not routed)
#pragma unroll
      for (int s = 0; s < CPS; ++s) b2s[s] = misc->bias[buf][s][t] * 1.4426950408889634f;   // -inf on padding rows
      const int kv0 = misc->kvbase[buf][0];
      ok = wait_on(bar(S_FULL + buf), (j >> 1) & 1);
      if (!ok) break;
      ptx::tc_fence_after();
      uint32_t sreg[64];
      {
        uint32_t* lo = sreg;
        uint32_t* hi = sreg + 32;
        DASH_TMEM_LD32(lo, lane_addr + buf * NKV);
        DASH_TMEM_LD32(hi, lane_addr + buf * NKV + 32);
      }
      ptx::tmem_wait_ld();

      // logit (log2 domain) = s*c1 + b2; c1 > 0, so the row maximum can be taken on the raw scores
      const int n_vis = i_row - kv0 + 1;             // causal: KV token kv0 + c visible iff c < n_vis
      bool selected;
      float mloc;
      if constexpr (CPS > 1) {
        // packed chunks: each slot of W columns has its own bias; only the own chunk (slot 0 of step 0) can be cut
        // by the causal mask (routed chunks lie wholly before the row)
        constexpr int W = NKV / CPS;
        mloc = -INFINITY;
#pragma unroll
        for (int s = 0; s < CPS; ++s) {
          if (b2s[s] > -INFINITY) {
            if (s == 0 && n_vis < W) {
#pragma unroll
              for (int c = 0; c < W; ++c)
                if (c >= n_vis) sreg[c] = 0xff800000u;   // -inf
            }
            float ch[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) ch[c] = __uint_as_float(sreg[s * W + c]);
#pragma unroll
            for (int k = 4; k < W; k += 4)
#pragma unroll
              for (int c = 0; c < 4; ++c) ch[c] = fmaxf(ch[c], __uint_as_float(sreg[s * W + c + k]));
            mloc = fmaxf(mloc, fmaf(fmaxf(fmaxf(ch[0], ch[1]), fmaxf(ch[2], ch[3])), c1, b2s[s]));
          }
        }
        selected = mloc > -INFINITY;
      }
      const float b2 = b2s[0];
      float mr = -INFINITY;
      if constexpr (CPS == 1) selected = b2 > -INFINITY;
      if (CPS == 1 && selected) {
        if (n_vis < NKV) {                           // only inside the own chunk
#pragma unroll
          for (int c = 0; c < NKV; ++c)
            if (c >= n_vis) sreg[c] = 0xff800000u;   // -inf
        }
        // three-input maxima: 32 instructions for the 64 scores, in eight independent chains, then a tree
        float ch[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) ch[c] = __uint_as_float(sreg[c]);
#pragma unroll
        for (int k = 8; k + 16 <= NKV; k += 16)
#pragma unroll
          for (int c = 0; c < 8; ++c) ch[c] = max3(ch[c], __uint_as_float(sreg[c + k]), __uint_as_float(sreg[c + k + 8]));
#pragma unroll
        for (int c = 0; c < 8; ++c) ch[c] = fmaxf(ch[c], __uint_as_float(sreg[c + NKV - 8]));
        mr = fmaxf(max3(ch[0], ch[1], ch[2]), fmaxf(max3(ch[3], ch[4], ch[5]), fmaxf(ch[6], ch[7])));
      }
      if constexpr (CPS == 1) mloc = fmaf(mr, c1, b2);           // -inf when not selected
      float corr = 1.f;
      bool moved = false;
      if (mloc > m_used + RESCALE_LOG2 || (m_used == -INFINITY && mloc > -INFINITY)) {
        corr = exp2f(m_used - mloc);   // 0 when nothing was accumulated yet
        m_used = mloc;
        moved = true;
      }
      l *= corr;
      [[maybe_unused]] uint32_t packed[STATS ? 1 : 32];
      if constexpr (STATS) {
        // P = hi + lo as two bf16 terms, 32 scores at a time, stored as they are formed (the scores are all in registers
        // already): hi into the first 32 columns of the step's S buffer, lo into the second 32
        float2 lsum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        const float2 c1v = make_float2(c1, c1);
        const float2 offv = make_float2(b2s[0] - m_used, b2s[0] - m_used);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t hi16[16], lo16[16];
          if (selected) {
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              const int cc = half * 32 + c;
              const float2 t = __ffma2_rn(make_float2(__uint_as_float(sreg[cc]), __uint_as_float(sreg[cc + 1])), c1v, offv);
              const float2 pp = make_float2(exp2f(t.x), exp2f(t.y));
              lsum[(c >> 1) & 1] = __fadd2_rn(lsum[(c >> 1) & 1], pp);
              __nv_bfloat162 h = __floats2bfloat162_rn(pp.x, pp.y);
              const float2 hf = __bfloat1622float2(h);
              __nv_bfloat162 lo = __floats2bfloat162_rn(pp.x - hf.x, pp.y - hf.y);
              hi16[c >> 1] = *reinterpret_cast<uint32_t*>(&h);
              lo16[c >> 1] = *reinterpret_cast<uint32_t*>(&lo);
            }
          } else {
#pragma unroll
            for (int c = 0; c < 16; ++c) hi16[c] = lo16[c] = 0u;
          }
          ptx::tmem_st_n<16>(lane_addr + buf * NKV + half * 16, hi16);
          ptx::tmem_st_n<16>(lane_addr + buf * NKV + 32 + half * 16, lo16);
        }
        const float2 ls = __fadd2_rn(lsum[0], lsum[1]);
        l += ls.x + ls.y;
      } else if (selected) {
        // scale-and-shift and the row sum on packed pairs (one instruction per two scores); a slot that is not
        // routed has offset -inf, so its probabilities come out as exactly 0
        const float2 c1v = make_float2(c1, c1);
        float2 offs[CPS];
#pragma unroll
        for (int s = 0; s < CPS; ++s) offs[s] = make_float2(b2s[s] - m_used, b2s[s] - m_used);
        float2 lsum[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
        for (int c = 0; c < NKV; c += 2) {
          const float2 offv = offs[c / (NKV / CPS)];
          const float2 t = __ffma2_rn(make_float2(__uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1])), c1v, offv);
          const float2 pp = make_float2(exp2f(t.x), exp2f(t.y));
          lsum[(c >> 1) & 3] = __fadd2_rn(lsum[(c >> 1) & 3], pp);
          __nv_bfloat162 h = __floats2bfloat162_rn(pp.x, pp.y);
          packed[c >> 1] = *reinterpret_cast<uint32_t*>(&h);
        }
        const float2 ls = __fadd2_rn(__fadd2_rn(lsum[0], lsum[1]), __fadd2_rn(lsum[2], lsum[3]));
        l += ls.x + ls.y;
      } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) packed[c] = 0u;
      }

      // O is stable once the previous step's PV has completed
      const bool fix = j > 0 && __any_sync(0xffffffffu, moved);
      if (fix) {
        ok = wait_on(bar(PV_DONE + (buf ^ 1)), ((j - 1) >> 1) & 1);
        if (!ok) break;
        ptx::tc_fence_after();
        // rescale this row of the accumulator: O *= 2^(m_old - m_new)
#pragma unroll 1
        for (int q = 0; q < HD / 32; ++q) {
          uint32_t o[32];
          DASH_TMEM_LD32(o, lane_addr + 2 * NKV + q * 32);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * corr);
          DASH_TMEM_ST32(lane_addr + 2 * NKV + q * 32, o);
        }
      }
      // P row -> the first 32 columns of this step's S buffer (two bf16 per column)
      if constexpr (!STATS) DASH_TMEM_ST32(lane_addr + buf * NKV, packed);
      ptx::tmem_wait_st();
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar(P_FULL + (j & 1)));
    }

    // epilogue: O / l -> global (row m is 128 contiguous bf16 of token i_row, head r*g_q + hh)
    if (ok && n_steps > 0) ok = wait_on(bar(PV_DONE + ((n_steps - 1) & 1)), ((n_steps - 1) >> 1) & 1);
    if (ok && n_steps > 0) {
      ptx::tc_fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const long long o_off = (long long)b * dm.os[0] + (long long)i_row * dm.os[1] + (long long)(r * g_q + hh) * dm.os[2];
      __nv_bfloat16* op = a.O + o_off;
      const bool row_out = i_row < dm.seq_q && (!SHORT || row_live);
      float dot = 0.f;
#pragma unroll 1
      for (int q = 0; q < HD / 32; ++q) {
        uint32_t o[32];
        DASH_TMEM_LD32(o, lane_addr + 2 * NKV + q * 32);
        ptx::tmem_wait_ld();
        if (STATS && row_out) {
          const __nv_bfloat16* gp = a.dO + o_off + q * 32;
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            const uint4 gv = *reinterpret_cast<const uint4*>(gp + c);
            const __nv_bfloat162* g2 = reinterpret_cast<const __nv_bfloat162*>(&gv);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const float2 gf = __bfloat1622float2(g2[u]);
              dot = fmaf(__uint_as_float(o[c + 2 * u]), gf.x, dot);
              dot = fmaf(__uint_as_float(o[c + 2 * u + 1]), gf.y, dot);
            }
          }
        }
        if (a.O && row_out) {
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            uint4 v;
            __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
            __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(o[c + 2]) * inv, __uint_as_float(o[c + 3]) * inv);
            __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(o[c + 4]) * inv, __uint_as_float(o[c + 5]) * inv);
            __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(o[c + 6]) * inv, __uint_as_float(o[c + 7]) * inv);
            v.x = *reinterpret_cast<uint32_t*>(&h0); v.y = *reinterpret_cast<uint32_t*>(&h1);
            v.z = *reinterpret_cast<uint32_t*>(&h2); v.w = *reinterpret_cast<uint32_t*>(&h3);
            *reinterpret_cast<uint4*>(op + q * 32 + c) = v;
          }
        }
      }
      if (STATS && row_out) {
        const long long row = (((long long)b * dm.h_kv + r) * a.n_tiles + tile) * 128 + m;
        a.lse2[row] = m_used + log2f(l);
        a.delta[row] = dot * inv;
      }
    }
    ptx::tc_fence_before();
  }

  __syncthreads();
  if (warp == 5) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, TMEM_COLS);
  }
  if (tid == 0 && misc->abort_flag) report_error(a.sb, DASH_ERR_TIMEOUT, 101);
}

// ---------------------------------------------------------------- host side

// [batch, tokens, heads, 128] bf16 tensor with element strides s[3]; box = 64 x box_heads x box_tokens x 1.
bool make_map(CUtensorMap* out, const void* base, int hd, long long tokens, int heads, int batch, const long long* s,
              int box_heads, int box_tokens) {
  cuuint64_t dims[4] = {(cuuint64_t)hd, (cuuint64_t)heads, (cuuint64_t)tokens, (cuuint64_t)batch};
  // a size-1 dimension may come with stride 0; any positive multiple of 16 bytes is accepted there
  auto st = [](long long e) { return (cuuint64_t)((e > 0 ? e : 8) * 2); };
  cuuint64_t strides[3] = {st(s[2]), st(s[1]), st(s[0])};
  cuuint32_t box[4] = {64u, (cuuint32_t)box_heads, (cuuint32_t)box_tokens, 1u};
  return encode_bf16_sw128_4d(out, base, dims, strides, box);
}

}  // namespace

bool prefill_sm100_supported(const Dims& dm) {
  if (dm.decode || !dm.causal || dm.dtype != DASH_BF16 || (dm.d != 64 && dm.d != 128)) return false;
  if (dm.B != 16 && dm.B != 32 && dm.B != 64 && dm.B != 128) return false;
  if (dm.g_q < 2 || 128 / dm.g_q > MAX_TQ) return false;
  if (dm.os[2] % 8 != 0 || dm.os[1] % 8 != 0) return false;
  return tensor_map_encoder() != nullptr;
}

cudaError_t launch_attend_prefill_sm100(const Dims& dm, const void* Q, const void* K, const void* V,
                                        const uint32_t* mask, const float* blk_bias, void* O, StatusBlock* sb,
                                        bool inputs_stable, cudaStream_t st, float* lse2, float* delta, const void* dO) {
  PrefillArgs a;
  a.lse2 = lse2;
  a.delta = delta;
  a.dO = (const __nv_bfloat16*)dO;
  a.dm = dm;
  a.TQ = 128 / dm.g_q < dm.B ? 128 / dm.g_q : dm.B;     // a tile stays inside one chunk
  a.n_tiles = (dm.seq_q + a.TQ - 1) / a.TQ;
  a.early_loads = inputs_stable ? 1 : 0;
  a.inject = test_hooks().skip_own_k_load;
  a.wait_limit = test_hooks().wait_limit_cycles;
  a.mask = mask;
  a.blk_bias = blk_bias;
  a.O = (__nv_bfloat16*)O;
  a.sb = sb;
  CUtensorMap tq, tk, tv;
  const int box_kv = dm.B < NKV ? dm.B : NKV;      // chunks below 64 tokens are fetched one box per chunk
  if (!make_map(&tq, Q, dm.d, dm.seq_q, dm.h_q, dm.batch, dm.qs, dm.g_q, a.TQ)) return cudaErrorInvalidValue;
  if (!make_map(&tk, K, dm.d, dm.seq_kv, dm.h_kv, dm.batch, dm.ks, 1, box_kv)) return cudaErrorInvalidValue;
  if (!make_map(&tv, V, dm.d, dm.seq_kv, dm.h_kv, dm.batch, dm.vs, 1, box_kv)) return cudaErrorInvalidValue;
  const long long blocks = (long long)a.n_tiles * dm.batch * dm.h_kv;
  cudaError_t le = cudaSuccess;
#define DASH_PF(HDV, CPSV, SHORTV)                                                                                  \
  {                                                                                                                 \
    static std::atomic<unsigned long long> configured{0};                                                           \
    if (cudaError_t e = allow_dynamic_smem(attend_prefill_sm100_kernel<HDV, CPSV, SHORTV>,                          \
                                           PfLayout<HDV, CPSV>::SMEM, configured);                                  \
        e != cudaSuccess)                                                                                           \
      return e;                                                                                                     \
    le = launch_chained(attend_prefill_sm100_kernel<HDV, CPSV, SHORTV>, dim3((unsigned)blocks), dim3(PF_THREADS),   \
                        PfLayout<HDV, CPSV>::SMEM, st, tq, tk, tv, a);                                              \
  }
#define DASH_PF_HD(HDV)                                                                    \
  if (cps == 1) DASH_PF(HDV, 1, false)                                                     \
  else if (cps == 2) { if (short_tile) DASH_PF(HDV, 2, true) else DASH_PF(HDV, 2, false) } \
  else { if (short_tile) DASH_PF(HDV, 4, true) else DASH_PF(HDV, 4, false) }
  const int cps = NKV / box_kv;
  const bool short_tile = a.TQ * dm.g_q < 128;      // only with chunks below 64 tokens
  if (lse2) {
    // statistics mode: the shapes the tensor-core backward takes (head_dim 128, chunks of 64 / 128, full tiles)
    if (dm.d != 128 || cps != 1 || short_tile || !delta || !dO) return cudaErrorInvalidValue;
    static std::atomic<unsigned long long> configured{0};
    if (cudaError_t e = allow_dynamic_smem(attend_prefill_sm100_kernel<128, 1, false, true>, PfLayout<128, 1>::SMEM, configured);
        e != cudaSuccess)
      return e;
    le = launch_chained(attend_prefill_sm100_kernel<128, 1, false, true>, dim3((unsigned)blocks), dim3(PF_THREADS),
                        PfLayout<128, 1>::SMEM, st, tq, tk, tv, a);
    count_launch();
    return le;
  }
  if (dm.d == 128) { DASH_PF_HD(128) } else { DASH_PF_HD(64) }
#undef DASH_PF_HD
#undef DASH_PF
  count_launch();
  return le;
}

}  // namespace dash
