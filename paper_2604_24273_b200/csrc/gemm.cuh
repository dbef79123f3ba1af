// a2+a3 for batched states (M > 16 tokens): the tensor-core kernel.
//
// The product is formed transposed, D[n, m] = sum_k C[n,k] * x_q[m,k], so that the ternary weights are the
// 128-row A operand and the tokens the (up to) 256-wide B operand of one tcgen05.mma: the 2-bit -> int8
// expansion, the only non-tensor work in the main loop, is then spent on the narrow side of the tile.
// C = W_q + 1 in {0,1,2} is fed as UNSIGNED bytes (decode = shift + mask), x_q as signed bytes; the surplus
// sum_k x_q[m,k] is subtracted in the epilogue.  All integer, exact.
//
// One persistent CTA per SM, 15 warps, three decoupled rings in shared memory:
//   warp 0      X producer : TMA tile of x_q (TOK tokens x 128 k, 128-byte swizzle)        ring of 128 KB
//   warp 2      P producer : bulk copy of the 4 KB packed weight piece (128 rows x 128 k)    ring of 8 x 4 KB
//   warps 3-6, 11-14 expand: packed piece -> int8 codes in the swizzled K-major layout       ring of 3 x 16 KB
//   warp 1      MMA        : the warp walks the loop, one elected lane issues tcgen05.mma kind::i8 (4 per k block,
//                            K = 32 each) into TMEM
//   warps 7-10  epilogue   : TMEM -> registers -> (acc - rowsum) * gamma*a_m/127 -> bf16/fp32, transposed through
//                            a per-warp shared-memory tile so that global stores are 16 bytes per lane
// The token-tile width TOK (64..256) is chosen per launch to fill the SMs with whole waves.
// Two 256-column accumulators in TMEM let the epilogue of tile i overlap the main loop of tile i+1.
// A variant for large launches pairs two CTAs of a cluster on a 256-row tile (tcgen05 cta_group::2, see PAIR below).
// Every mbarrier wait is bounded; on expiry the CTA records a status word and leaves through the normal exit.
#pragma once

#include <cuda.h>

#include "clsk.cuh"
#include "common.cuh"
#include "ptx.cuh"

namespace bitrl {

constexpr int GM_ROWS = 128;  // weight rows per tile  (MMA M)
constexpr int GM_TOK_MAX = 256;  // tokens per tile (MMA N) is a template parameter: 64, 128, 192 or 256
constexpr int GM_BK = 128;    // k per pipeline stage  (one 128-byte swizzle row of int8)
constexpr uint32_t GM_X_RING_BYTES = 131072;  // x_q ring: as many (tokens x 128 k) stages as fit in 128 KB
constexpr int GM_PS = 8;      // packed-weight ring depth
constexpr int GM_WS = 3;      // expanded-weight ring depth
constexpr int GM_THREADS = 480;  // 15 warps: 3 single-thread roles, 2 x 4 expander warps, 4 epilogue warps
constexpr int GM_EXPAND2_WARP0 = 11;  // second expander group
constexpr int GM_EXPAND_WARP0 = 3;
constexpr int GM_EPI_WARP0 = 7;

constexpr uint32_t GM_W_BYTES = GM_ROWS * GM_BK;  // 16384
constexpr uint32_t GM_P_BYTES = TILE_BYTES;       // 4096
constexpr uint32_t GM_STAGE_BYTES = 2048;         // per epilogue warp: 32 tokens x 32 rows bf16 (or 16 x 32 fp32)
constexpr uint32_t GM_OFF_X = 0;
constexpr uint32_t GM_OFF_W = GM_OFF_X + GM_X_RING_BYTES;
constexpr uint32_t GM_OFF_P = GM_OFF_W + GM_WS * GM_W_BYTES;
constexpr uint32_t GM_OFF_STAGE = GM_OFF_P + GM_PS * GM_P_BYTES;
constexpr uint32_t GM_OFF_TOK = GM_OFF_STAGE + 4 * GM_STAGE_BYTES;  // scale[2][256] f32, rowsum[2][256] i32
constexpr uint32_t GM_OFF_BAR = GM_OFF_TOK + 2 * GM_TOK_MAX * 8;
constexpr uint32_t GM_XS_MAX = 16;
constexpr uint32_t GM_NUM_BARS = 2 * GM_XS_MAX + 2 * GM_PS + 2 * GM_WS + 4;
constexpr uint32_t GM_OFF_MISC = GM_OFF_BAR + GM_NUM_BARS * 8;
constexpr uint32_t GM_SMEM_BYTES = GM_OFF_MISC + 32 + 1024;  // + slack to align the base to 1024
static_assert(GM_SMEM_BYTES <= 232448, "shared memory budget of one CTA");

// stage ids reported with BITRL_ERR_TIMEOUT
enum { GM_WAIT_X_EMPTY = 1, GM_WAIT_P_EMPTY = 2, GM_WAIT_P_FULL = 3, GM_WAIT_W_EMPTY = 4, GM_WAIT_TMEM_EMPTY = 5,
       GM_WAIT_X_FULL = 6, GM_WAIT_W_FULL = 7, GM_WAIT_TMEM_FULL = 8 };

struct GemmArgs {
  const uint8_t* tiles;
  const float* gamma;
  const float* absmax;
  const int32_t* rowsum;
  int M, N, K;
  void* y;
  int out_dtype;
  const unsigned short* residual;
  int32_t* acc_out;
  int tiles_n, tiles_total;
  // Split-K for launches with few tiles: work item = (tile, k range); the raw int32 partial sums of an item are added
  // into `part` [M,N] (zeroed by the launcher) with integer atomics - exact and order-free - and a second kernel applies
  // the epilogue.  splits == 1: one item per tile, epilogue in this kernel, `part` unused.
  int splits, kb_per_split;
  int32_t* part;
};

// PAIR: two CTAs of a cluster work on one 256-row x TOK-token tile with tcgen05.mma.cta_group::2.  CTA rank r expands
// weight rows [256 t + 128 r, +128) into its own tensor memory, fetches tokens [TOK/2 * r, +TOK/2) of the tile into its
// own shared memory and drains its own 128 x TOK slice of the accumulator; rank 0 issues the MMAs.  Per SM this halves
// the B-operand traffic through shared memory, the binding resource of the single-CTA kernel.  The barriers that gate
// the MMA (x_full, tmem_empty) are rank 0's and collect the arrivals of both CTAs; the barriers that the MMA's
// completion releases (x_empty, tmem_full) exist in both CTAs and are reached by one multicast commit.
//
// CLSK (cluster split-K, for launches with few tiles): the a.splits CTAs of a cluster take the k ranges of ONE tile, one
// item per CTA.  When its main loop is done a CTA sends, through distributed shared memory, every peer the raw int32
// partial sums of the token columns that peer owns (columns are dealt in units of 8, unit range [r U / S, (r+1) U / S)
// to rank r); after one cluster barrier each CTA adds what it received to its own partial sums and applies the
// epilogue to its columns.  Integer sums: exact and independent of the order, so the result equals the unsplit one.
template <int GM_TOK, bool A_TMEM, bool PAIR = false, bool CLSK = false>
__global__ void __launch_bounds__(GM_THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap tmap_x, const GemmArgs a) {
  static_assert(!PAIR || A_TMEM, "the paired kernel keeps its weights in tensor memory");
  static_assert(!PAIR || GM_TOK % 16 == 0, "each CTA holds TOK/2 tokens in whole 8-row swizzle groups");
  static_assert(!CLSK || (A_TMEM && !PAIR && GM_TOK <= 128), "cluster split-K: narrow single-CTA tiles, weights in tensor memory");
  constexpr uint32_t GM_X_BYTES = (PAIR ? GM_TOK / 2 : GM_TOK) * GM_BK;  // this CTA's part of a token tile
  // x_q ring: 128 KB, plus the 48 KB of the shared-memory weight ring when the weights go through tensor memory
  // (4 stages at 256 tokens, 6 at 224, 7 at 192, 11 at 128, 16 at 64).  The cluster split-K variant takes the end of
  // that area for the partial sums it receives from its peers.
  constexpr uint32_t GM_RECV = CLSK ? clsk_recv_bytes(GM_TOK) : 0u;
  constexpr uint32_t GM_X_RING = A_TMEM ? GM_OFF_P - GM_OFF_X - GM_RECV : GM_X_RING_BYTES;
  constexpr uint32_t GM_XS = GM_X_RING / GM_X_BYTES < GM_XS_MAX ? GM_X_RING / GM_X_BYTES : GM_XS_MAX;
  static_assert(GM_TOK % 32 == 0 && GM_TOK >= 64 && GM_TOK <= GM_TOK_MAX && GM_XS <= GM_XS_MAX, "token tile");
  // With the A operand in tensor memory the two accumulators sit at columns [0,TOK) and [256,256+TOK).
  // Weight slots in tensor memory are the 32-column pieces between the end of each accumulator and the next multiple
  // of 256: slot i sits behind accumulator (i & 1), piece i / 2.  TOK = 224 leaves two slots, TOK <= 192 four.
#ifndef GM_WSK_CAP
#define GM_WSK_CAP 12
#endif
  constexpr uint32_t WSK_FREE = 2 * ((256 - GM_TOK) / 32);  // every free 32-column piece of tensor memory is a slot
  constexpr uint32_t WSK_CAP = GM_WSK_CAP < GM_XS - 1 ? GM_WSK_CAP : GM_XS - 1;
  constexpr uint32_t WSK = !A_TMEM ? GM_WS : (WSK_FREE < WSK_CAP ? WSK_FREE : WSK_CAP);
  static_assert(!A_TMEM || (GM_TOK <= 224 && WSK >= 2), "tensor-memory column budget");
  static_assert(WSK < GM_XS, "the expanders watch the x_q ring WSK steps behind; a watched barrier must not flip twice");
  auto a_slot = [](uint32_t slot) { return (slot & 1u) * 256u + GM_TOK + 32u * (slot >> 1); };
  extern __shared__ unsigned char gm_smem_raw[];
  const uint32_t raw_addr = ptx::smem_u32(gm_smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* base_ptr = gm_smem_raw + (base - raw_addr);

  const uint32_t bar_x_full = base + GM_OFF_BAR;
  const uint32_t bar_x_empty = bar_x_full + 8 * GM_XS;
  const uint32_t bar_p_full = bar_x_empty + 8 * GM_XS;
  const uint32_t bar_p_empty = bar_p_full + 8 * GM_PS;
  const uint32_t bar_w_full = bar_p_empty + 8 * GM_PS;
  const uint32_t bar_w_empty = bar_w_full + 8 * GM_WS;
  const uint32_t bar_tmem_full = bar_w_empty + 8 * GM_WS;  // [2]
  const uint32_t bar_tmem_empty = bar_tmem_full + 16;      // [2]
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + GM_OFF_MISC);
  // Set by the first role whose wait ran out of time (in both CTAs of a pair).  Every wait polls it, so the other
  // roles stop within a few hundred polls instead of each waiting out its own limit, and the teardown drains.
  volatile uint32_t* failed = reinterpret_cast<volatile uint32_t*>(base_ptr + GM_OFF_MISC + 8);
  const uint32_t failed_addr = base + GM_OFF_MISC + 8;
  const uint32_t bar_drain = base + GM_OFF_MISC + 16;  // only used on the failure path

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kblocks = a.K / GM_BK;
  const int items = a.tiles_total * a.splits;
  // PAIR: both CTAs of a cluster walk the same items (tiles_n then counts 256-row tiles); rank selects the halves.
  const uint32_t rank = (PAIR || CLSK) ? ptx::cluster_ctarank() : 0u;  // CLSK: = the item's k range (clusters are consecutive CTAs)
  const uint32_t recv_base = base + GM_OFF_P - GM_RECV;
  const uint32_t failed_peer = PAIR ? ptx::mapa_u32(failed_addr, rank ^ 1u) : 0u;
  auto wait = [&](uint32_t bar, uint32_t parity) { return ptx::mbar_wait_abortable(bar, parity, failed_addr); };
  auto give_up = [&](int stage) {
    report_timeout(stage);
    *failed = 1u;
    if (PAIR) asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(failed_peer), "r"(1u) : "memory");
  };
  const int item0 = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int item_step = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
  const uint32_t x_full_lead = PAIR ? ptx::mapa_u32(bar_x_full, 0) : bar_x_full;        // as seen from either CTA
  const uint32_t tmem_empty_lead = PAIR ? ptx::mapa_u32(bar_tmem_empty, 0) : bar_tmem_empty;
  auto item_range = [&](int item, int& tile, int& kb0, int& kb1) {
    tile = item / a.splits;
    kb0 = (item - tile * a.splits) * a.kb_per_split;
    kb1 = min(kblocks, kb0 + a.kb_per_split);
  };

  if (threadIdx.x == 0) {
    *failed = 0u;
    ptx::mbar_init(bar_drain, 1);
    // x_full: the producer's expect_tx arrival plus one arrival per expander warp (of both CTAs when paired)
    for (int s = 0; s < GM_XS; ++s) {
      ptx::mbar_init(bar_x_full + 8 * s, PAIR ? 1 + 8 : 1 + 4);
      ptx::mbar_init(bar_x_empty + 8 * s, 1);
    }
    for (int s = 0; s < GM_PS; ++s) { ptx::mbar_init(bar_p_full + 8 * s, 1); ptx::mbar_init(bar_p_empty + 8 * s, 4); }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(bar_tmem_full + 8 * b, 1);
      ptx::mbar_init(bar_tmem_empty + 8 * b, PAIR ? 8 : 4);
    }
    ptx::mbar_init_fence();
    ptx::tma_prefetch_desc(&tmap_x);
  }
  if (warp == 1) {
    if (PAIR) {
      ptx::tmem_alloc_pair(base + GM_OFF_MISC, 512);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(base + GM_OFF_MISC, 512);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  // the peer's barriers are initialised (PAIR) / every CTA of the cluster has started (CLSK) before anything is sent to it
  if (PAIR || CLSK) ptx::cluster_sync_all();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // Barriers and tensor memory are set up: the next kernel in the stream may start its own set-up.  Only the roles that
  // touch what the preceding kernel wrote (the x_q producer; the epilogue: scales, row sums, residual, outputs) wait for
  // it; the packed weights are constant, so their copies, the expansion into tensor memory and everything else that
  // does not need x_q start while the predecessor is still draining.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    // ------------------------------------------------------------------ X producer
    if (lane == 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      uint32_t it = 0;
      bool ok = true;
      for (int item = item0; ok && item < items; item += item_step) {
        int tile, kb0, kb1;
        item_range(item, tile, kb0, kb1);
        const int tm = tile / a.tiles_n;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const uint32_t s = it % GM_XS, ph = (it / GM_XS) & 1u;
          if (!wait(bar_x_empty + 8 * s, ph ^ 1u)) { give_up(GM_WAIT_X_EMPTY); ok = false; break; }
          if (PAIR) {
            // Rank 0 announces the bytes of both halves on its barrier; each CTA's copy reports there.
            if (rank == 0) ptx::mbar_arrive_expect_tx(bar_x_full + 8 * s, 2 * GM_X_BYTES);
            ptx::tma_load_2d_pair(base + GM_OFF_X + s * GM_X_BYTES, &tmap_x, kb * GM_BK,
                                  tm * GM_TOK + static_cast<int>(rank) * (GM_TOK / 2), x_full_lead + 8 * s);
          } else {
            ptx::mbar_arrive_expect_tx(bar_x_full + 8 * s, GM_X_BYTES);
            ptx::tma_load_2d(base + GM_OFF_X + s * GM_X_BYTES, &tmap_x, kb * GM_BK, tm * GM_TOK, bar_x_full + 8 * s);
          }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ P producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int item = item0; ok && item < items; item += item_step) {
        int tile, kb0, kb1;
        item_range(item, tile, kb0, kb1);
        const int tn = PAIR ? 2 * (tile % a.tiles_n) + static_cast<int>(rank) : tile % a.tiles_n;
        const uint8_t* wsrc = a.tiles + static_cast<size_t>(tn) * kblocks * TILE_BYTES;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const uint32_t s = it % GM_PS, ph = (it / GM_PS) & 1u;
          if (!wait(bar_p_empty + 8 * s, ph ^ 1u)) { give_up(GM_WAIT_P_EMPTY); ok = false; break; }
          ptx::mbar_arrive_expect_tx(bar_p_full + 8 * s, GM_P_BYTES);
          ptx::bulk_g2s(base + GM_OFF_P + s * GM_P_BYTES, wsrc + static_cast<size_t>(kb) * TILE_BYTES, GM_P_BYTES,
                        bar_p_full + 8 * s);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp walks the loop (waits included) and one elected lane issues: with uniform control flow the
    // descriptors and addresses stay in uniform registers, which is what the MMA instruction takes its operands from.
    if (!PAIR || rank == 0) {
      const uint32_t idesc = ptx::idesc_i8(PAIR ? 2 * GM_ROWS : GM_ROWS, GM_TOK, /*a_signed=*/false, /*b_signed=*/true);
      uint32_t lt = 0;
      uint32_t xs = 0, xph = 0, ws = 0;  // ring slots and phase, advanced without divisions
      bool ok = true;
      for (int item = item0; ok && item < items; item += item_step, ++lt) {
        int tile, kb0, kb1;
        item_range(item, tile, kb0, kb1);
        const uint32_t buf = lt & 1u;
        if (!__any_sync(0xffffffffu, wait(bar_tmem_empty + 8 * buf, ((lt >> 1) & 1u) ^ 1u))) {
          if (lane == 0) give_up(GM_WAIT_TMEM_EMPTY);
          ok = false;
          break;
        }
        const uint32_t d_tmem = tmem_base + buf * GM_TOK_MAX;
        ptx::tc_fence_after_sync();  // orders this tile's MMAs after the epilogue's reads of the accumulator
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!__any_sync(0xffffffffu, wait(bar_x_full + 8 * xs, xph))) {
            if (lane == 0) give_up(GM_WAIT_X_FULL);
            ok = false;
            break;
          }
          // Weights written with tcgen05.st by other threads need the tcgen05 fence on this side of the barrier;
          // TMA data and expander stores to shared memory (already fenced into the async proxy by their writers) do not.
          if (A_TMEM) ptx::tc_fence_after_sync();
          const uint64_t bdesc = ptx::smem_desc_sw128(base + GM_OFF_X + xs * GM_X_BYTES);
          if (ptx::elect_one()) {
          if (PAIR) {
            const uint32_t a_tmem = tmem_base + a_slot(ws);
#pragma unroll
            for (int k4 = 0; k4 < GM_BK / 32; ++k4)
              ptx::mma_i8_ts_pair(d_tmem, a_tmem + 8 * k4, bdesc + 2 * k4, idesc, (kb != kb0 || k4 != 0) ? 1u : 0u);
          } else if (A_TMEM) {
            const uint32_t a_tmem = tmem_base + a_slot(ws);
#pragma unroll
            for (int k4 = 0; k4 < GM_BK / 32; ++k4)
              ptx::mma_i8_ts(d_tmem, a_tmem + 8 * k4, bdesc + 2 * k4, idesc, (kb != kb0 || k4 != 0) ? 1u : 0u);
          } else {
            const uint64_t adesc = ptx::smem_desc_sw128(base + GM_OFF_W + ws * GM_W_BYTES);
#pragma unroll
            for (int k4 = 0; k4 < GM_BK / 32; ++k4)
              ptx::mma_i8_ss(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kb != kb0 || k4 != 0) ? 1u : 0u);
          }
          // frees the x_q slot and the weight slot of this k block (in both CTAs of a pair)
          if (PAIR) ptx::mma_commit_pair(bar_x_empty + 8 * xs, 3);
          else ptx::mma_commit(bar_x_empty + 8 * xs);
          }
          __syncwarp();
          if (++xs == GM_XS) { xs = 0; xph ^= 1u; }
          if (++ws == WSK) ws = 0;
        }
        if (ok && ptx::elect_one()) {
          if (PAIR) ptx::mma_commit_pair(bar_tmem_full + 8 * buf, 3);
          else ptx::mma_commit(bar_tmem_full + 8 * buf);
        }
        __syncwarp();
      }
    }
  } else if (warp < GM_EPI_WARP0 || warp >= GM_EXPAND2_WARP0) {
    // ------------------------------------------------------------------ expanders (one weight row each)
    // Two groups of four warps alternate k blocks (group 0 the even ones, group 1 the odd ones): one group needs
    // longer for a block than the tensor pipe does, two keep ahead of it.
    const uint32_t grp = warp >= GM_EXPAND2_WARP0 ? 1u : 0u;
    // Shared-memory A: any thread may expand any row.  Tensor-memory A: a warp can only write its own lane quarter
    // (warp id mod 4), so its 32 lanes take the 32 rows of that quarter.
    const int r = A_TMEM ? (warp & 3) * 32 + lane
                         : static_cast<int>(threadIdx.x) - (grp ? GM_EXPAND2_WARP0 : GM_EXPAND_WARP0) * 32;
    const uint32_t row_off = static_cast<uint32_t>(r >> 3) * 1024u + static_cast<uint32_t>(r & 7) * 128u;
    const uint32_t sw = static_cast<uint32_t>(r & 7);
    // The weight slot of k block `it` was last used by k block it - WSK; that MMA's completion is the arrival on
    // x_empty of ITS x_q slot, so the expanders watch the x_q ring WSK steps behind (WSK < GM_XS keeps the
    // watched barrier at most one phase ahead).  Their "ready" arrival goes to x_full of the current x_q slot, which
    // therefore completes when both the TMA bytes and the four expander warps are in: one wait per k block for the MMA.
    uint32_t it = 0;
    uint32_t ps = 0, pph = 0, ws = 0, xs = 0, xs_old = 0, xph_old = 0;
    bool ok = true;
    for (int item = item0; ok && item < items; item += item_step) {
      int tile, kb0, kb1;
      item_range(item, tile, kb0, kb1);
      for (int kb = kb0; kb < kb1; ++kb, ++it) {
        if ((it & 1u) != grp) {  // the other group's k block: only advance the ring positions
          if (it >= WSK && ++xs_old == GM_XS) { xs_old = 0; xph_old ^= 1u; }
          if (++ps == GM_PS) { ps = 0; pph ^= 1u; }
          if (++ws == WSK) ws = 0;
          if (++xs == GM_XS) xs = 0;
          continue;
        }
        // All lanes poll the same barrier; a phase that one lane saw complete is complete, so the vote makes the
        // outcome warp-uniform (the tcgen05.st below is a whole-warp instruction).
        if (!__any_sync(0xffffffffu, wait(bar_p_full + 8 * ps, pph))) {
          if (lane == 0) give_up(GM_WAIT_P_FULL);
          ok = false;
          break;
        }
        const uint32_t paddr = base + GM_OFF_P + ps * GM_P_BYTES + r * TILE_ROW_BYTES;
        const uint4 p0 = ptx::lds128(paddr), p1 = ptx::lds128(paddr + 16);
        if (it >= WSK) {
          if (!__any_sync(0xffffffffu, wait(bar_x_empty + 8 * xs_old, xph_old))) {
            if (lane == 0) give_up(GM_WAIT_W_EMPTY);
            ok = false;
            break;
          }
          if (++xs_old == GM_XS) { xs_old = 0; xph_old ^= 1u; }
        }
        if (A_TMEM) ptx::tc_fence_after_sync();
        const uint32_t wd[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
        if (A_TMEM) {
          // row r, k = 4c..4c+3 -> 32-bit column c of TMEM lane r: the whole 128-k slice is one 32-column store
          uint32_t cols[32];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            cols[4 * j + 0] = wd[j] & 0x03030303u;
            cols[4 * j + 1] = (wd[j] >> 2) & 0x03030303u;
            cols[4 * j + 2] = (wd[j] >> 4) & 0x03030303u;
            cols[4 * j + 3] = (wd[j] >> 6) & 0x03030303u;
          }
          ptx::tmem_st_32x32b_x32(tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16) +
                                      a_slot(ws), cols);
          ptx::tmem_st_wait();
          ptx::tc_fence_before_sync();
        } else {
          const uint32_t wrow = base + GM_OFF_W + ws * GM_W_BYTES + row_off;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            uint4 c;
            c.x = wd[j] & 0x03030303u;
            c.y = (wd[j] >> 2) & 0x03030303u;
            c.z = (wd[j] >> 4) & 0x03030303u;
            c.w = (wd[j] >> 6) & 0x03030303u;
            ptx::sts128(wrow + ((static_cast<uint32_t>(j) ^ sw) << 4), c);
          }
          ptx::fence_proxy_async_smem();
        }
        __syncwarp();
        if (lane == 0) {
          if (PAIR) ptx::mbar_arrive_cluster(x_full_lead + 8 * xs);
          else ptx::mbar_arrive(bar_x_full + 8 * xs);
          ptx::mbar_arrive(bar_p_empty + 8 * ps);
        }
        if (++ps == GM_PS) { ps = 0; pph ^= 1u; }
        if (++ws == WSK) ws = 0;
        if (++xs == GM_XS) xs = 0;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int q = warp & 3;                           // TMEM lane quarter this warp may read
    const int ep = threadIdx.x - GM_EPI_WARP0 * 32;   // 0..127
    const int ew = warp - GM_EPI_WARP0;               // staging buffer index
    const uint32_t stage = base + GM_OFF_STAGE + ew * GM_STAGE_BYTES;
    const float gamma = *a.gamma;
    const bool f32 = a.out_dtype == BITRL_OUT_F32;
    uint32_t lt = 0;
    bool ok = true;
    if constexpr (CLSK) {
      // One item per CTA: exchange of the partial sums inside the cluster, then the epilogue on this CTA's columns.
      const int tile = static_cast<int>(blockIdx.x) / a.splits;
      const ClskArgs c{tmem_base, recv_base, base + GM_OFF_TOK, base + GM_OFF_TOK + 2 * GM_TOK_MAX * 4, rank, a.splits,
                       tile % a.tiles_n, tile / a.tiles_n, a.M, a.N, gamma, a.absmax, a.rowsum, a.y, a.out_dtype,
                       a.residual, a.acc_out, failed};
      if (!clsk_exchange_epilogue<GM_TOK>(c, q, lane, ep, [&] { return wait(bar_tmem_full, 0u); }) && ep == 0)
        give_up(GM_WAIT_TMEM_FULL);
      (void)lt; (void)ok; (void)stage; (void)ew; (void)f32;
    } else
    for (int item = item0; ok && item < items; item += item_step, ++lt) {
      const int tile = item / a.splits;
      const int tn = PAIR ? 2 * (tile % a.tiles_n) + static_cast<int>(rank) : tile % a.tiles_n, tm = tile / a.tiles_n;
      const uint32_t buf = lt & 1u;
      const uint32_t sc_addr = base + GM_OFF_TOK + buf * GM_TOK_MAX * 4;
      const uint32_t rs_addr = base + GM_OFF_TOK + 2 * GM_TOK_MAX * 4 + buf * GM_TOK_MAX * 4;
      for (int j = ep; j < GM_TOK; j += 128) {
        const int tok = tm * GM_TOK + j;
        ptx::sts32(sc_addr + 4 * j, __float_as_uint(tok < a.M ? out_scale(gamma, a.absmax[tok]) : 0.0f));
        ptx::sts32(rs_addr + 4 * j, static_cast<uint32_t>(tok < a.M ? a.rowsum[tok] : 0));
      }
      // The named barrier that publishes the scales also ANDs the outcome of the wait over the four epilogue warps, so
      // that they either all go on (to whole-warp tensor-memory loads and the next round of this barrier) or all leave.
      if (!ptx::bar_red_and(1, 128, wait(bar_tmem_full + 8 * buf, (lt >> 1) & 1u))) {
        if (ep == 0) give_up(GM_WAIT_TMEM_FULL);
        ok = false;
        break;
      }
      ptx::tc_fence_after_sync();
      const int nbase = tn * GM_ROWS + q * 32;  // first output column of this warp
      const int tok0 = tm * GM_TOK;
      const int tok_hi = min(GM_TOK, a.M - tok0);
      for (int c = 0; c < GM_TOK / 32; ++c) {
        if (c * 32 >= tok_hi) break;  // warp-uniform
        // Residual rows of this chunk are requested first, so their latency hides behind the accumulator load, the
        // rescale and the transpose (in-place updates make every later store a possible alias for the compiler).
        uint4 rres[4];
        if (a.residual && !f32) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int t = i * 8 + (lane >> 2);
            if (c * 32 + t < tok_hi)
              rres[i] = ptx::ldg128(a.residual + static_cast<size_t>(tok0 + c * 32 + t) * a.N + nbase + (lane & 3) * 8);
          }
        }
        uint32_t v[32];
        ptx::tmem_ld_32x32b_x32(tmem_base + buf * GM_TOK_MAX + c * 32 + (static_cast<uint32_t>(q * 32) << 16), v);
        ptx::tmem_ld_wait();
        if (a.part) {  // split-K item: hand the raw partial sums over, the finishing kernel does the rest
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c * 32 + j < tok_hi)
              atomicAdd(a.part + static_cast<size_t>(tok0 + c * 32 + j) * a.N + nbase + lane, static_cast<int>(v[j]));
          continue;
        }
        // acc = D - rowsum (exact int32), y = acc * scale
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const uint4 rs4 = ptx::lds128(rs_addr + (c * 32 + 4 * g) * 4);
          v[4 * g + 0] -= rs4.x; v[4 * g + 1] -= rs4.y; v[4 * g + 2] -= rs4.z; v[4 * g + 3] -= rs4.w;
        }
        if (a.acc_out) {  // debug tap, plain stores
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c * 32 + j < tok_hi)
              a.acc_out[static_cast<size_t>(tok0 + c * 32 + j) * a.N + nbase + lane] = static_cast<int>(v[j]);
        }
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const uint4 sc4 = ptx::lds128(sc_addr + (c * 32 + 4 * g) * 4);
          v[4 * g + 0] = __float_as_uint(__fmul_rn(static_cast<float>(static_cast<int>(v[4 * g + 0])), __uint_as_float(sc4.x)));
          v[4 * g + 1] = __float_as_uint(__fmul_rn(static_cast<float>(static_cast<int>(v[4 * g + 1])), __uint_as_float(sc4.y)));
          v[4 * g + 2] = __float_as_uint(__fmul_rn(static_cast<float>(static_cast<int>(v[4 * g + 2])), __uint_as_float(sc4.z)));
          v[4 * g + 3] = __float_as_uint(__fmul_rn(static_cast<float>(static_cast<int>(v[4 * g + 3])), __uint_as_float(sc4.w)));
        }
        if (!f32) {
          // transpose 32 tokens x 32 columns of bf16 through shared memory: row = token (64 bytes)
#pragma unroll
          for (int j = 0; j < 32; ++j) ptx::sts16(stage + j * 64 + lane * 2, float_to_bf16_bits(__uint_as_float(v[j])));
          __syncwarp();
          unsigned short* yb = static_cast<unsigned short*>(a.y);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int t = i * 8 + (lane >> 2), part = lane & 3;
            uint4 o = ptx::lds128(stage + i * 512 + lane * 16);
            if (c * 32 + t < tok_hi) {
              const size_t off = static_cast<size_t>(tok0 + c * 32 + t) * a.N + nbase + part * 8;
              if (a.residual) {
                const uint4 rr = rres[i];
                const uint32_t ov[4] = {o.x, o.y, o.z, o.w}, rv[4] = {rr.x, rr.y, rr.z, rr.w};
                uint32_t res[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const float lo = __fadd_rn(__uint_as_float(rv[e] << 16), __uint_as_float(ov[e] << 16));
                  const float hi = __fadd_rn(__uint_as_float(rv[e] & 0xffff0000u), __uint_as_float(ov[e] & 0xffff0000u));
                  res[e] = static_cast<uint32_t>(float_to_bf16_bits(lo)) | (static_cast<uint32_t>(float_to_bf16_bits(hi)) << 16);
                }
                o = make_uint4(res[0], res[1], res[2], res[3]);
              }
              *reinterpret_cast<uint4*>(yb + off) = o;
            }
          }
          __syncwarp();
        } else {
          // fp32: two passes of 16 tokens x 32 columns (row = token, 128 bytes)
          float* yf = static_cast<float*>(a.y);
#pragma unroll
          for (int h = 0; h < 2; ++h) {
#pragma unroll
            for (int j = 0; j < 16; ++j) ptx::sts32(stage + j * 128 + lane * 4, v[h * 16 + j]);
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int t = h * 16 + i * 4 + (lane >> 3), part = lane & 7;
              const uint4 o = ptx::lds128(stage + i * 512 + lane * 16);
              if (c * 32 + t < tok_hi)
                *reinterpret_cast<uint4*>(yf + static_cast<size_t>(tok0 + c * 32 + t) * a.N + nbase + part * 4) = o;
            }
            __syncwarp();
          }
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) ptx::mbar_arrive_cluster(tmem_empty_lead + 8 * buf);
        else ptx::mbar_arrive(bar_tmem_empty + 8 * buf);
      }
    }
  }

  // ---- teardown: every role leaves through here, also after a timeout ----
  __syncwarp();
  ptx::tc_fence_before_sync();
  if constexpr (CLSK) {
    // the cluster barrier of the exchange: the epilogue warps pass it inside their role, everyone else here
    if (warp < GM_EPI_WARP0 || warp >= GM_EXPAND2_WARP0) ptx::cluster_sync_all();
  }
  __syncthreads();
  if (PAIR) ptx::cluster_sync_all();  // neither CTA leaves (or frees tensor memory) while the other may still reach it
  if (*failed) {
    // Failure path only: a role gave up, so copies and MMAs that nobody waited for may still be in flight.  The MMA
    // issuer waits (bounded) for its MMAs, then every thread lets about a millisecond pass, far longer than any copy
    // takes, before shared and tensor memory are given back.
    if (warp == 1 && (!PAIR || rank == 0)) {
      if (ptx::elect_one()) {
        if (PAIR) ptx::mma_commit_pair(bar_drain, 1);
        else ptx::mma_commit(bar_drain);
      }
      __syncwarp();
      ptx::mbar_wait(bar_drain, 0, 2000000LL);
    }
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {}
    __syncthreads();
    if (PAIR) ptx::cluster_sync_all();  // `failed` is the same in both CTAs after the first cluster barrier
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    if (PAIR) ptx::tmem_dealloc_pair(tmem_base, 512);
    else ptx::tmem_dealloc(tmem_base, 512);
  }
}

// cuTensorMapEncodeTiled, resolved through the runtime so the library does not link against libcuda.
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline encode_tiled_fn get_encode_tiled() {
  static encode_tiled_fn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<encode_tiled_fn>(p);
  }
  return fn;
}

int sm_count();
bool gemm_a_in_tmem();
int gemm_pair_mode();     // BITRL_GEMM_PAIR: 1 = paired CTAs wherever the shape allows, 0 = never, unset = launcher's choice
int gemm_clsk_mode();     // BITRL_GEMM_CLSK: 0 = no cluster split-K (the scratch + finishing-kernel form is used instead)
int gemm_forced_tok();    // 0, or the token-tile width forced through BITRL_GEMM_TOK (64, 128, 192, 224, 256)  // expanded weights through tensor memory (default) or through shared memory

// Second kernel of a split-K launch: y = (part - rowsum) * gamma * a_m / 127 (+ residual), 8 outputs per thread.
__global__ void __launch_bounds__(256) gemm_splitk_finish_kernel(const int32_t* part, const float* gamma, const float* absmax,
                                                               const int32_t* rowsum, int M, int N, void* y, int out_dtype,
                                                               const unsigned short* residual, int32_t* acc_out) {
  pdl_enter();
  const int n8 = N >> 3;
  const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<long long>(M) * n8) return;
  const int m = static_cast<int>(idx / n8);
  const size_t off = static_cast<size_t>(idx) * 8;
  const uint4 p0 = *reinterpret_cast<const uint4*>(part + off), p1 = *reinterpret_cast<const uint4*>(part + off + 4);
  const int rs = rowsum[m];
  const float scale = out_scale(*gamma, absmax[m]);
  const int acc[8] = {static_cast<int>(p0.x) - rs, static_cast<int>(p0.y) - rs, static_cast<int>(p0.z) - rs,
                      static_cast<int>(p0.w) - rs, static_cast<int>(p1.x) - rs, static_cast<int>(p1.y) - rs,
                      static_cast<int>(p1.z) - rs, static_cast<int>(p1.w) - rs};
  if (acc_out) {
    *reinterpret_cast<int4*>(acc_out + off) = make_int4(acc[0], acc[1], acc[2], acc[3]);
    *reinterpret_cast<int4*>(acc_out + off + 4) = make_int4(acc[4], acc[5], acc[6], acc[7]);
  }
  float v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = __fmul_rn(static_cast<float>(acc[e]), scale);
  if (out_dtype == BITRL_OUT_F32) {
    float* yf = static_cast<float*>(y) + off;
    *reinterpret_cast<float4*>(yf) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(yf + 4) = make_float4(v[4], v[5], v[6], v[7]);
    return;
  }
  uint32_t o[4];
  uint4 rr = make_uint4(0u, 0u, 0u, 0u);
  if (residual) rr = *reinterpret_cast<const uint4*>(residual + off);
  const uint32_t rv[4] = {rr.x, rr.y, rr.z, rr.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    unsigned short lo = float_to_bf16_bits(v[2 * e]), hi = float_to_bf16_bits(v[2 * e + 1]);
    if (residual) {
      lo = float_to_bf16_bits(__fadd_rn(__uint_as_float(rv[e] << 16), bf16_bits_to_float(lo)));
      hi = float_to_bf16_bits(__fadd_rn(__uint_as_float(rv[e] & 0xffff0000u), bf16_bits_to_float(hi)));
    }
    o[e] = static_cast<uint32_t>(lo) | (static_cast<uint32_t>(hi) << 16);
  }
  *reinterpret_cast<uint4*>(static_cast<unsigned short*>(y) + off) = make_uint4(o[0], o[1], o[2], o[3]);
}

// Paired-CTA launches are considered from this M on (many tiles, no split-K).  A sweep of the five block shapes showed
// pairs never ahead at M = 1024 and 2048 (equal to 3 us behind) and ahead on four of five at M = 4096.
constexpr int GM_PAIR_MIN_M = 3072;
constexpr int GM_PAIR_FORCED_MIN_M = 1024;  // with BITRL_GEMM_PAIR=1 (tests of the paired kernel on small ragged shapes)

// Time per k block (ns) of one CTA (or CTA pair) by token-tile width, as measured at M = 4096 on the block shapes: the
// 192-wide tile runs close to the tensor pipe's own time; at 224 only two weight slots fit beside the accumulators in
// tensor memory and the expand -> MMA -> release chain shows; at 256 the weights go through shared memory, whose
// bandwidth then binds; below 192 the fixed cost per k block (barrier round trips, issue) is the floor.
inline long long gemm_kb_ns(int tok, bool pair) {
  if (pair) return tok == 224 ? 340 : tok == 192 ? 283 : 284;
  return tok == 256 ? 466 : tok == 224 ? 372 : tok == 192 ? 295 : tok == 128 ? 284 : 270;
}

inline void (*gemm_pair_kernel(int tok))(const CUtensorMap, const GemmArgs) {
  return tok == 224 ? gemm_i8_kernel<224, true, true> : tok == 192 ? gemm_i8_kernel<192, true, true>
                                                                   : gemm_i8_kernel<128, true, true>;
}

// Clusters of two CTAs that can be resident at once (the persistent grid must not exceed it), per device and width.
inline int gemm_pair_max_clusters(int tok) {
  static int cached[64][3] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  const int slot = tok == 224 ? 0 : tok == 192 ? 1 : 2;
  if (cached[dev][slot] == 0) {
    void (*pk)(const CUtensorMap, const GemmArgs) = gemm_pair_kernel(tok);
    int n = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * 74);
    cfg.blockDim = dim3(GM_THREADS);
    cfg.dynamicSmemBytes = GM_SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(pk, cudaFuncAttributeMaxDynamicSharedMemorySize, GM_SMEM_BYTES) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, pk, &cfg) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = -1;
    }
    cached[dev][slot] = n;
  }
  if (cached[dev][slot] > 0) return cached[dev][slot];
  // The occupancy query can fail under a profiler.  When the paired kernel is forced (BITRL_GEMM_PAIR=1) fall back to
  // one cluster per SM pair: the grid is a static partition of the tiles, CTAs wait only on their own cluster peer, so
  // a grid larger than what is resident at once is merely queued.
  return gemm_pair_mode() == 1 ? sm_count() / 2 : 0;
}

inline void (*gemm_clsk_kernel(int tok))(const CUtensorMap, const GemmArgs) {
  return tok == 128 ? gemm_i8_kernel<128, true, false, true> : gemm_i8_kernel<64, true, false, true>;
}

// Clusters of `S` CTAs of the cluster split-K kernel that can be resident at once (0: this size cannot be launched).
inline int gemm_clsk_max_clusters(int tok, int S) {
  static int cached[64][2][9] = {};
  int dev = 0;
  if (S < 2 || S > 8 || cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  int& c = cached[dev][tok == 128 ? 1 : 0][S];
  if (c == 0) {
    void (*k)(const CUtensorMap, const GemmArgs) = gemm_clsk_kernel(tok);
    int n = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S * 32);
    cfg.blockDim = dim3(GM_THREADS);
    cfg.dynamicSmemBytes = GM_SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, GM_SMEM_BYTES) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, k, &cfg) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = -1;
    }
    c = n;
  }
  if (c > 0) return c;
  // The query can fail under a profiler.  The grid is a static partition and a CTA waits only for the peers of its own
  // cluster, so an optimistic count merely queues clusters; sizes that may not exist at all are not offered then.
  return (S == 2 || S == 4 || S == 8) ? sm_count() / S : 0;
}

// Largest M for which a split-K workspace (M*N int32) is offered.
constexpr int GM_SPLITK_MAX_M = 512;

// What the launcher does with an [M, K] x [N, K] product on the current device.
struct GemmPlan {
  int tok, splits;    // token-tile width; k ranges per tile
  bool clsk, pair;    // splits > 1 reduced inside a cluster (else through scratch); 256-row tiles on CTA pairs
  int pair_clusters;  // persistent grid of the paired kernel
};

// have_ws: the caller offers M*N int32 of scratch (the scratch form of split-K needs it).
inline GemmPlan gemm_plan(int N, int K, int M, bool have_ws) {
  // Token-tile width and split count: fewest "waves x k blocks per item x time per k block" over the SMs.
  const int sms = sm_count();
  const int tiles_n = N / GM_ROWS;
  const int kblocks = K / GM_BK;
  int tok = 256, splits = 1;
  bool clsk = false;  // split over the CTAs of a cluster (reduced through distributed shared memory) or through scratch
  long long best = -1;
  {
    const int cand[5] = {256, 224, 192, 128, 64};
    for (int i = 0; i < 5; ++i) {
      if (cand[i] == 224 && !gemm_a_in_tmem()) continue;
      const long long tiles = static_cast<long long>(tiles_n) * ((M + cand[i] - 1) / cand[i]);
      const long long per_kb = gemm_kb_ns(cand[i], false);
      const int smax = (have_ws && M <= GM_SPLITK_MAX_M && tiles * 2 <= sms) ? static_cast<int>(sms / tiles) : 1;
      for (int sp = 1; sp <= smax && sp <= kblocks; ++sp) {
        const int kps = (kblocks + sp - 1) / sp;
        if ((kblocks + kps - 1) / kps != sp) continue;  // this count would leave an empty split
        const long long waves = (tiles * sp + sms - 1) / sms;
        // a split launch pays for clearing the scratch and for the finishing kernel (about 5 us in a chain of dependent launches)
        const long long cost = waves * kps * per_kb + (sp > 1 ? 5000 : 0);
        if (best < 0 || cost <= best) { best = cost; tok = cand[i]; splits = sp; clsk = false; }  // ties go to the narrower tile
      }
      // Cluster split-K needs no scratch and no further launch.  Measured against the unsplit kernel (M = 32 ... 256 on
      // the block shapes) a wave of clusters costs 1.5 - 2.5 us more than its k blocks: the cluster launch (growing with
      // the number of clusters), two cluster barriers and the exchange (growing with the cluster size).
      if (cand[i] <= 128 && tiles * 2 <= sms && gemm_clsk_mode() != 0 && gemm_a_in_tmem()) {
        for (int sp = 2; sp <= 8 && sp <= kblocks; ++sp) {
          const int kps = (kblocks + sp - 1) / sp;
          if ((kblocks + kps - 1) / kps != sp) continue;
          if (!clsk_fits(cand[i], sp)) continue;
          const int clusters = gemm_clsk_max_clusters(cand[i], sp);
          if (clusters <= 0) continue;
          long long cost = ((tiles + clusters - 1) / clusters) * (kps * per_kb + 1500 + 150 * sp + 15 * tiles);
          if (gemm_clsk_mode() == sp) cost = 0;  // forced size (tuning knob); the narrowest tile that allows it wins
          if (cost <= best) { best = cost; tok = cand[i]; splits = sp; clsk = true; }
        }
      }
    }
  }
  if (const int forced = gemm_forced_tok()) { tok = forced; splits = 1; clsk = false; }  // tuning knob, see bitrl.cu
  // CTA pairs (256-row tiles): for launches with many tiles, an even number of 128-row tiles and weights in tensor memory.
  bool pair = false;
  int pair_clusters = 0;
  if (gemm_pair_mode() != 0 && gemm_a_in_tmem() && tiles_n % 2 == 0 && splits == 1 &&
      M >= (gemm_pair_mode() == 1 ? GM_PAIR_FORCED_MIN_M : GM_PAIR_MIN_M)) {
    int ptok = 0;
    if (const int forced = gemm_forced_tok()) {
      if (forced == 224 || forced == 192 || forced == 128) ptok = forced;
    } else {
      long long pbest = -1;
      const int cand[3] = {224, 192, 128};
      for (int i = 0; i < 3; ++i) {
        const int clusters = gemm_pair_max_clusters(cand[i]);
        if (clusters <= 0) continue;
        const long long tiles = static_cast<long long>(tiles_n / 2) * ((M + cand[i] - 1) / cand[i]);
        // a cluster launch starts and ends a little later than a plain one; 1.5 us reproduces the measured choices at
        // M = 4096 (pairs at 224 tokens for 2560 -> 3840 / 6912 / 13824, at 192 for 6912 -> 2560, single CTAs for 2560 -> 2560)
        const long long cost = ((tiles + clusters - 1) / clusters) * kblocks * gemm_kb_ns(cand[i], true) + 1500;
        if (pbest < 0 || cost < pbest) { pbest = cost; ptok = cand[i]; }
      }
      if (gemm_pair_mode() != 1 && pbest >= best) ptok = 0;  // the single-CTA kernel is expected to be no slower
    }
    if (ptok) {
      pair_clusters = gemm_pair_max_clusters(ptok);
      if (pair_clusters > 0) { pair = true; tok = ptok; }
    }
  }
  return GemmPlan{tok, splits, clsk, pair, pair_clusters};
}

// splitk_ws: nullptr, or M*N int32 of scratch that allows the scratch form of split-K when the launch has too few
// tiles to fill the SMs and the cluster form does not apply.
bitrl_status launch_gemm(const Linear* w, const int8_t* xq, const float* absmax, const int32_t* rowsum, int M,
                         void* y, int out_dtype, const void* residual, int32_t* acc_out, cudaStream_t st,
                         int32_t* splitk_ws) {
  encode_tiled_fn encode = get_encode_tiled();
  if (!encode) return cuda_fail(cudaErrorSymbolNotFound);
  const GemmPlan plan = gemm_plan(w->N, w->K, M, splitk_ws != nullptr);
  const int sms = sm_count();
  const int tiles_n = w->N / GM_ROWS;
  const int kblocks = w->K / GM_BK;
  const int tok = plan.tok, splits = plan.splits, pair_clusters = plan.pair_clusters;
  const bool clsk = plan.clsk, pair = plan.pair;
  CUtensorMap tmap;
  const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(w->K), static_cast<cuuint64_t>(M)};
  const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(w->K)};
  const cuuint32_t box[2] = {GM_BK, static_cast<cuuint32_t>(pair ? tok / 2 : tok)};  // a paired CTA fetches half a tile
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(xq), gdim, gstride, box,
                            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cuda_fail(cudaErrorInvalidValue);

  if (clsk) {
    GemmArgs a{w->tiles, w->gamma, absmax, rowsum, M, w->N, w->K, y, out_dtype, static_cast<const unsigned short*>(residual),
               acc_out, tiles_n, tiles_n * ((M + tok - 1) / tok), splits, (kblocks + splits - 1) / splits, nullptr};
    void (*ck)(const CUtensorMap, const GemmArgs) = gemm_clsk_kernel(tok);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(a.tiles_total * splits));  // cluster c = tile c, rank = k range
    cfg.blockDim = dim3(GM_THREADS);
    cfg.dynamicSmemBytes = GM_SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(splits);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    BITRL_CUDA(cudaFuncSetAttribute(ck, cudaFuncAttributeMaxDynamicSharedMemorySize, GM_SMEM_BYTES));
    BITRL_CUDA(cudaLaunchKernelEx(&cfg, ck, tmap, a));
    count_launch(1);
    return BITRL_OK;
  }
  const bool split = splits > 1;
  GemmArgs a{w->tiles, w->gamma, absmax, rowsum, M, w->N, w->K, y, out_dtype,
             split ? nullptr : static_cast<const unsigned short*>(residual), split ? nullptr : acc_out, tiles_n, 0,
             splits, (kblocks + splits - 1) / splits, split ? splitk_ws : nullptr};
  if (pair) {
    a.tiles_n = tiles_n / 2;
    a.tiles_total = a.tiles_n * ((M + tok - 1) / tok);
    const int clusters = a.tiles_total < pair_clusters ? a.tiles_total : pair_clusters;
    void (*pk)(const CUtensorMap, const GemmArgs) = gemm_pair_kernel(tok);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * clusters);
    cfg.blockDim = dim3(GM_THREADS);
    cfg.dynamicSmemBytes = GM_SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    BITRL_CUDA(cudaLaunchKernelEx(&cfg, pk, tmap, a));
    count_launch(1);
    return BITRL_OK;
  }
  a.tiles_total = tiles_n * ((M + tok - 1) / tok);
  const int items = a.tiles_total * splits;
  const int grid = items < sms ? items : sms;
  if (split) BITRL_CUDA(cudaMemsetAsync(splitk_ws, 0, static_cast<size_t>(M) * w->N * sizeof(int32_t), st));
  const bool a_tmem = gemm_a_in_tmem() && tok <= 224;
  void (*kern)(const CUtensorMap, const GemmArgs) =
      tok == 256 ? gemm_i8_kernel<256, false>
      : tok == 224 ? gemm_i8_kernel<224, true>
      : tok == 192 ? (a_tmem ? gemm_i8_kernel<192, true> : gemm_i8_kernel<192, false>)
      : tok == 128 ? (a_tmem ? gemm_i8_kernel<128, true> : gemm_i8_kernel<128, false>)
                   : (a_tmem ? gemm_i8_kernel<64, true> : gemm_i8_kernel<64, false>);
  BITRL_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, GM_SMEM_BYTES));
  BITRL_CUDA(launch_pdl(kern, dim3(grid), dim3(GM_THREADS), GM_SMEM_BYTES, st, tmap, a));
  count_launch(1);
  if (split) {
    const long long n = static_cast<long long>(M) * (w->N / 8);
    BITRL_CUDA(launch_pdl(gemm_splitk_finish_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, st,
                          static_cast<const int32_t*>(splitk_ws), w->gamma, absmax, rowsum, M, w->N, y, out_dtype,
                          static_cast<const unsigned short*>(residual), acc_out));
    count_launch(1);
  }
  return BITRL_OK;
}

}  // namespace bitrl
