// W8A8 layer for the higher-precision critic backbone (Sec. V ablations, Table IV: "INT8 critic + 1-bit policy"):
// the same int8 activation quantization and int32 contraction as the ternary layer, with int8 weights (one symmetric
// absmax scale per matrix).  There is nothing to decode, so both operands of tcgen05.mma kind::i8 come straight from
// TMA tiles in shared memory: D[n, m] = sum_k W_q[n,k] * x_q[m,k], weights the 128-row A operand (signed), tokens the
// TOK-wide B operand (signed).
//
// One persistent CTA per SM, 6 warps:
//   warp 0      producer: per k block one TMA tile of W_q (128 rows x 128 k) and one of x_q (TOK tokens x 128 k),
//               both 128-byte swizzled, on one barrier
//   warp 1      MMA: one thread issues four K=32 instructions per k block into one of two TMEM accumulators
//   warps 2-5   epilogue: TMEM -> registers -> (float)acc * scale_w * a_m / 127 -> bf16/fp32, transposed through a
//               per-warp shared-memory tile for 16-byte stores; overlaps the next tile's main loop
// Every mbarrier wait is bounded; on expiry the CTA records a status word and leaves through the normal exit.
#pragma once

#include <cuda.h>

#include "clsk.cuh"
#include "common.cuh"
#include "gemm.cuh"
#include "gemv.cuh"
#include "ptx.cuh"

namespace bitrl {

constexpr int G8_THREADS = 192;
constexpr int G8_EPI_WARP0 = 2;
constexpr uint32_t G8_W_BYTES = 128 * 128;
constexpr uint32_t G8_RING_BYTES = 196608;
constexpr uint32_t G8_MAX_STAGES = 8;
constexpr uint32_t G8_OFF_STAGE = G8_RING_BYTES;                      // 4 x 2 KB epilogue tiles
constexpr uint32_t G8_OFF_TOK = G8_OFF_STAGE + 4 * 2048;              // scale[2][256] f32
constexpr uint32_t G8_OFF_BAR = G8_OFF_TOK + 2 * 256 * 4;
constexpr uint32_t G8_OFF_MISC = G8_OFF_BAR + (2 * G8_MAX_STAGES + 4) * 8;
constexpr uint32_t G8_SMEM_BYTES = G8_OFF_MISC + 32 + 1024;           // + slack to align the base to 1024
static_assert(G8_SMEM_BYTES <= 232448, "shared memory budget of one CTA");

constexpr int G8_PAIR_MIN_M = 2048;  // paired CTAs from this M on
enum { G8_WAIT_EMPTY = 41, G8_WAIT_FULL = 42, G8_WAIT_TMEM_EMPTY = 43, G8_WAIT_TMEM_FULL = 44 };

struct Gemm8Args {
  const float* scale;   // [1] weight scale
  const float* absmax;  // [M]
  int M, N, K;
  void* y;
  int out_dtype;
  const unsigned short* residual;
  int32_t* acc_out;
  int tiles_n, tiles_total;
  int splits, kb_per_split;  // cluster split-K (CLSK below): k ranges per tile; 1 and K/128 otherwise
};

// PAIR: two CTAs of a cluster work on one 256-row x TOK-token tile with tcgen05.mma.cta_group::2, as in the ternary
// GEMM: rank r fetches weight rows [256 t + 128 r, +128) and tokens [TOK/2 * r, +TOK/2) of the tile into its own
// shared memory (completion counted on rank 0's barrier) and drains its own 128 x TOK slice of the accumulator;
// rank 0 issues the MMAs and releases the stage in both CTAs with one multicast commit.  Per SM the B tile is halved,
// and shared-memory traffic is what binds this kernel.
//
// CLSK (launches with few tiles): the a.splits CTAs of a cluster take the k ranges of ONE tile, one item per CTA, and
// exchange their int32 partial sums through distributed shared memory (clsk.cuh); the receive area is the end of the ring.
template <int TOK, bool PAIR = false, bool CLSK = false>
__global__ void __launch_bounds__(G8_THREADS, 1)
gemm_w8_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w, const Gemm8Args a) {
  static_assert(!CLSK || (!PAIR && TOK <= 128), "cluster split-K: narrow single-CTA tiles");
  constexpr uint32_t X_BYTES = (PAIR ? TOK / 2 : TOK) * 128;
  constexpr uint32_t STAGE = X_BYTES + G8_W_BYTES;
  constexpr uint32_t RECV = CLSK ? clsk_recv_bytes(TOK) : 0u;
  constexpr uint32_t NS = (G8_RING_BYTES - RECV) / STAGE < G8_MAX_STAGES ? (G8_RING_BYTES - RECV) / STAGE : G8_MAX_STAGES;
  static_assert(TOK % 32 == 0 && TOK >= 64 && TOK <= 256, "token tile");
  extern __shared__ unsigned char g8_smem_raw[];
  const uint32_t raw_addr = ptx::smem_u32(g8_smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* base_ptr = g8_smem_raw + (base - raw_addr);
  const uint32_t bar_full = base + G8_OFF_BAR;
  const uint32_t bar_empty = bar_full + 8 * G8_MAX_STAGES;
  const uint32_t bar_tmem_full = bar_empty + 8 * G8_MAX_STAGES;  // [2]
  const uint32_t bar_tmem_empty = bar_tmem_full + 16;            // [2]
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + G8_OFF_MISC);
  // Set by the first role whose wait ran out of time (in both CTAs of a pair); every wait polls it.
  volatile uint32_t* failed = reinterpret_cast<volatile uint32_t*>(base_ptr + G8_OFF_MISC + 8);
  const uint32_t failed_addr = base + G8_OFF_MISC + 8;
  const uint32_t bar_drain = base + G8_OFF_MISC + 16;  // only used on the failure path

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kblocks = a.K / 128;
  const uint32_t rank = (PAIR || CLSK) ? ptx::cluster_ctarank() : 0u;  // CLSK: = the k range (clusters are consecutive CTAs)
  const int tile0 = CLSK ? static_cast<int>(blockIdx.x) / a.splits
                         : PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int tile_step = CLSK ? a.tiles_total : PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
  const int kb0 = CLSK ? static_cast<int>(rank) * a.kb_per_split : 0;
  const int kb1 = CLSK ? min(kblocks, kb0 + a.kb_per_split) : kblocks;
  const uint32_t full_lead = PAIR ? ptx::mapa_u32(bar_full, 0) : bar_full;  // rank 0's barriers as seen from either CTA
  const uint32_t tmem_empty_lead = PAIR ? ptx::mapa_u32(bar_tmem_empty, 0) : bar_tmem_empty;
  const uint32_t failed_peer = PAIR ? ptx::mapa_u32(failed_addr, rank ^ 1u) : 0u;
  auto wait = [&](uint32_t bar, uint32_t parity) { return ptx::mbar_wait_abortable(bar, parity, failed_addr); };
  auto give_up = [&](int stage) {
    report_timeout(stage);
    *failed = 1u;
    if (PAIR) asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(failed_peer), "r"(1u) : "memory");
  };

  if (threadIdx.x == 0) {
    *failed = 0u;
    ptx::mbar_init(bar_drain, 1);
    for (uint32_t s = 0; s < NS; ++s) { ptx::mbar_init(bar_full + 8 * s, 1); ptx::mbar_init(bar_empty + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(bar_tmem_full + 8 * b, 1);
      ptx::mbar_init(bar_tmem_empty + 8 * b, PAIR ? 8 : 4);
    }
    ptx::mbar_init_fence();
    ptx::tma_prefetch_desc(&tmap_x);
    ptx::tma_prefetch_desc(&tmap_w);
  }
  if (warp == 1) {
    if (PAIR) {
      ptx::tmem_alloc_pair(base + G8_OFF_MISC, 512);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(base + G8_OFF_MISC, 512);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  // the peer's barriers are initialised (PAIR) / every CTA of the cluster has started (CLSK) before anything is sent to it
  if (PAIR || CLSK) ptx::cluster_sync_all();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  pdl_enter();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t s = 0, ph = 0;
      bool ok = true;
      for (int tile = tile0; ok && tile < a.tiles_total; tile += tile_step) {
        const int tn = PAIR ? 2 * (tile % a.tiles_n) + static_cast<int>(rank) : tile % a.tiles_n, tm = tile / a.tiles_n;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!wait(bar_empty + 8 * s, ph ^ 1u)) { give_up(G8_WAIT_EMPTY); ok = false; break; }
          if (PAIR) {
            // Rank 0 announces the bytes of both CTAs' stages on its barrier; each CTA's copies report there.
            if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full + 8 * s, 2 * STAGE);
            ptx::tma_load_2d_pair(base + s * STAGE, &tmap_w, kb * 128, tn * 128, full_lead + 8 * s);
            ptx::tma_load_2d_pair(base + s * STAGE + G8_W_BYTES, &tmap_x, kb * 128,
                                  tm * TOK + static_cast<int>(rank) * (TOK / 2), full_lead + 8 * s);
            if (++s == NS) { s = 0; ph ^= 1u; }
            continue;
          }
          ptx::mbar_arrive_expect_tx(bar_full + 8 * s, STAGE);
          ptx::tma_load_2d(base + s * STAGE, &tmap_w, kb * 128, tn * 128, bar_full + 8 * s);
          ptx::tma_load_2d(base + s * STAGE + G8_W_BYTES, &tmap_x, kb * 128, tm * TOK, bar_full + 8 * s);
          if (++s == NS) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp walks the loop and one elected lane issues: uniform control flow keeps the descriptors in
    // uniform registers, from which the MMA instruction takes its operands.
    if (!PAIR || rank == 0) {
      const uint32_t idesc = ptx::idesc_i8(PAIR ? 256 : 128, TOK, /*a_signed=*/true, /*b_signed=*/true);
      uint32_t s = 0, ph = 0, lt = 0;
      bool ok = true;
      for (int tile = tile0; ok && tile < a.tiles_total; tile += tile_step, ++lt) {
        const uint32_t buf = lt & 1u;
        if (!__any_sync(0xffffffffu, wait(bar_tmem_empty + 8 * buf, ((lt >> 1) & 1u) ^ 1u))) {
          if (lane == 0) give_up(G8_WAIT_TMEM_EMPTY);
          ok = false;
          break;
        }
        const uint32_t d_tmem = tmem_base + buf * 256;
        ptx::tc_fence_after_sync();
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!__any_sync(0xffffffffu, wait(bar_full + 8 * s, ph))) {
            if (lane == 0) give_up(G8_WAIT_FULL);
            ok = false;
            break;
          }
          const uint64_t adesc = ptx::smem_desc_sw128(base + s * STAGE);
          const uint64_t bdesc = ptx::smem_desc_sw128(base + s * STAGE + G8_W_BYTES);
          if (ptx::elect_one()) {
            if (PAIR) {
#pragma unroll
              for (int k4 = 0; k4 < 4; ++k4)
                ptx::mma_i8_ss_pair(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kb != kb0 || k4 != 0) ? 1u : 0u);
              ptx::mma_commit_pair(bar_empty + 8 * s, 3);  // frees the stage in both CTAs
            } else {
#pragma unroll
              for (int k4 = 0; k4 < 4; ++k4)
                ptx::mma_i8_ss(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kb != kb0 || k4 != 0) ? 1u : 0u);
              ptx::mma_commit(bar_empty + 8 * s);
            }
          }
          __syncwarp();
          if (++s == NS) { s = 0; ph ^= 1u; }
        }
        if (ok && ptx::elect_one()) {
          if (PAIR) ptx::mma_commit_pair(bar_tmem_full + 8 * buf, 3);
          else ptx::mma_commit(bar_tmem_full + 8 * buf);
        }
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    const int ep = threadIdx.x - G8_EPI_WARP0 * 32;  // 0..127
    const int ew = warp - G8_EPI_WARP0;
    const uint32_t stage = base + G8_OFF_STAGE + ew * 2048;
    const float wscale = *a.scale;
    const bool f32 = a.out_dtype == BITRL_OUT_F32;
    uint32_t lt = 0;
    bool ok = true;
    if constexpr (CLSK) {
      // One item per CTA: exchange of the partial sums inside the cluster, then the epilogue on this CTA's columns.
      const ClskArgs c{tmem_base, base + G8_RING_BYTES - RECV, base + G8_OFF_TOK, base + G8_OFF_TOK + 256 * 4, rank,
                       a.splits, tile0 % a.tiles_n, tile0 / a.tiles_n, a.M, a.N, wscale, a.absmax, nullptr, a.y,
                       a.out_dtype, a.residual, a.acc_out, failed};
      if (!clsk_exchange_epilogue<TOK>(c, q, lane, ep, [&] { return wait(bar_tmem_full, 0u); }) && ep == 0)
        give_up(G8_WAIT_TMEM_FULL);
      (void)lt; (void)ok; (void)stage; (void)ew; (void)f32;
    } else
    for (int tile = tile0; ok && tile < a.tiles_total; tile += tile_step, ++lt) {
      const int tn = PAIR ? 2 * (tile % a.tiles_n) + static_cast<int>(rank) : tile % a.tiles_n, tm = tile / a.tiles_n;
      const uint32_t buf = lt & 1u;
      const uint32_t sc_addr = base + G8_OFF_TOK + buf * 256 * 4;
      for (int j = ep; j < TOK; j += 128) {
        const int tok = tm * TOK + j;
        ptx::sts32(sc_addr + 4 * j, __float_as_uint(tok < a.M ? out_scale(wscale, a.absmax[tok]) : 0.0f));
      }
      // The named barrier that publishes the scales also ANDs the outcome of the wait over the four epilogue warps:
      // they all go on (whole-warp tensor-memory loads, the next round of this barrier) or all leave.
      if (!ptx::bar_red_and(1, 128, wait(bar_tmem_full + 8 * buf, (lt >> 1) & 1u))) {
        if (ep == 0) give_up(G8_WAIT_TMEM_FULL);
        ok = false;
        break;
      }
      ptx::tc_fence_after_sync();
      const int nbase = tn * 128 + q * 32;
      const int tok0 = tm * TOK;
      const int tok_hi = min(TOK, a.M - tok0);
      for (int c = 0; c < TOK / 32; ++c) {
        if (c * 32 >= tok_hi) break;  // warp-uniform
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
        ptx::tmem_ld_32x32b_x32(tmem_base + buf * 256 + c * 32 + (static_cast<uint32_t>(q * 32) << 16), v);
        ptx::tmem_ld_wait();
        if (a.acc_out) {
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
    // the cluster barrier of the exchange: the epilogue warps pass it inside their role, the other two warps here
    if (warp < G8_EPI_WARP0) ptx::cluster_sync_all();
  }
  __syncthreads();
  if (PAIR) ptx::cluster_sync_all();  // neither CTA leaves (or frees tensor memory) while the other may still reach it
  if (*failed) {
    // Failure path only: copies and MMAs that nobody waited for may still be in flight.  The MMA issuer waits (bounded)
    // for its MMAs, then every thread lets about a millisecond pass before shared and tensor memory are given back.
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

inline void (*gemm_w8_pair_kernel(int tok))(const CUtensorMap, const CUtensorMap, const Gemm8Args) {
  return tok == 256 ? gemm_w8_kernel<256, true> : tok == 192 ? gemm_w8_kernel<192, true> : gemm_w8_kernel<128, true>;
}

// Clusters of two CTAs that can be resident at once, per device and width (0 = paired launches unavailable).
inline int gemm_w8_pair_max_clusters(int tok) {
  static int cached[64][3] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  const int slot = tok == 256 ? 0 : tok == 192 ? 1 : 2;
  if (cached[dev][slot] == 0) {
    void (*pk)(const CUtensorMap, const CUtensorMap, const Gemm8Args) = gemm_w8_pair_kernel(tok);
    int n = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * 74);
    cfg.blockDim = dim3(G8_THREADS);
    cfg.dynamicSmemBytes = G8_SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(pk, cudaFuncAttributeMaxDynamicSharedMemorySize, G8_SMEM_BYTES) != cudaSuccess ||
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

inline void (*gemm_w8_clsk_kernel(int tok))(const CUtensorMap, const CUtensorMap, const Gemm8Args) {
  return tok == 128 ? gemm_w8_kernel<128, false, true> : gemm_w8_kernel<64, false, true>;
}

// Clusters of `S` CTAs of the cluster split-K kernel that can be resident at once (0: this size cannot be launched).
inline int gemm_w8_clsk_max_clusters(int tok, int S) {
  static int cached[64][2][9] = {};
  int dev = 0;
  if (S < 2 || S > 8 || cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  int& c = cached[dev][tok == 128 ? 1 : 0][S];
  if (c == 0) {
    void (*k)(const CUtensorMap, const CUtensorMap, const Gemm8Args) = gemm_w8_clsk_kernel(tok);
    int n = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S * 32);
    cfg.blockDim = dim3(G8_THREADS);
    cfg.dynamicSmemBytes = G8_SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, G8_SMEM_BYTES) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, k, &cfg) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = -1;
    }
    c = n;
  }
  if (c > 0) return c;
  return (S == 2 || S == 4 || S == 8) ? sm_count() / S : 0;  // the query can fail under a profiler (see gemm.cuh)
}

// ---- M <= 16: streaming kernel ----------------------------------------------------------------------------------
// The weights (N*K bytes) are read once; the kernel is bound by HBM.  Persistent CTAs of 8 warps: the activations are
// quantized once per CTA into shared memory (one warp per token), then a warp owns a few weight rows at a time, every
// lane streams 16-byte pieces of them and feeds dp4a (signed x signed) for all tokens; one shuffle tree per row.
constexpr int GV8_THREADS = 256;

struct Gemv8Args {
  const int8_t* wq;
  const float* scale;
  const unsigned short* x;  // bf16 [M,K]
  int M, N, K;
  void* y;
  int out_dtype;
  int8_t* xq_out;      // debug taps (may be null)
  float* absmax_out;
  int32_t* acc_out;
};

__device__ __forceinline__ int dp4a_s8s8(uint32_t a, uint32_t b, int acc) {
  int d;
  asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(acc));
  return d;
}

template <int MT, int R>
__global__ void __launch_bounds__(GV8_THREADS) gemv_w8_kernel(Gemv8Args a) {
  extern __shared__ __align__(16) unsigned char gv8_smem[];
  int8_t* xq_s = reinterpret_cast<int8_t*>(gv8_smem);               // [MT][K]
  float* sc_s = reinterpret_cast<float*>(gv8_smem + MT * a.K);      // [MT] a_m / 127
  __shared__ float redf[GV8_THREADS / 32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = a.K, nvec8 = K >> 3, nvec16 = K >> 4;
  // A warp streams R rows at a time (N is a multiple of 128): R times as many loads in flight per lane, and every
  // 16-byte piece of the activations read from shared memory serves R rows.  The launcher takes fewer rows per warp
  // when the matrix has too few rows to give every SM a CTA otherwise.
  constexpr int PRE = 2;  // 16-byte steps of the first row group requested before anything else
  const int n_first = (blockIdx.x * (GV8_THREADS / 32) + warp) * R;
  // The weights depend neither on the activations nor on the preceding kernel: the first loads of this warp's first
  // rows are in flight while the CTA waits for its predecessor and quantizes the activations.
  uint4 pre[PRE][R];
  if (n_first < a.N) {
    const uint4* wr = reinterpret_cast<const uint4*>(a.wq + static_cast<size_t>(n_first) * K);
#pragma unroll
    for (int p = 0; p < PRE; ++p)
#pragma unroll
      for (int r = 0; r < R; ++r)
        if (lane + 32 * p < nvec16) pre[p][r] = __ldg(wr + static_cast<size_t>(r) * nvec16 + lane + 32 * p);
  }
  pdl_enter();
  // Activations: WPR warps share a token (all eight for one token), largest magnitude through shared memory.
  constexpr int NW = GV8_THREADS / 32;
  constexpr int WPR = MT >= NW ? 1 : NW / MT;
  constexpr int RPP = NW / WPR;
  const int sub = warp % WPR;
#pragma unroll 1
  for (int pass = 0; pass < (MT + RPP - 1) / RPP; ++pass) {
    const int m = pass * RPP + warp / WPR;
    const bool live = m < a.M;
    uint2* dst = reinterpret_cast<uint2*>(xq_s + (m < MT ? m : 0) * K);
    const uint4* xr = reinterpret_cast<const uint4*>(a.x + static_cast<size_t>(live ? m : 0) * K);
    float mx = 0.0f;
    if (live) {
#pragma unroll 4
      for (int i = sub * 32 + lane; i < nvec8; i += WPR * 32) mx = fmaxf(mx, absmax8(xr[i]));
    }
    mx = warp_max(mx);
    if (WPR > 1) {
      if (lane == 0) redf[warp] = mx;
      __syncthreads();
#pragma unroll
      for (int i = 0; i < WPR; ++i) mx = fmaxf(mx, redf[(warp / WPR) * WPR + i]);
      __syncthreads();
    }
    const float amax = fmaxf(mx, 1e-5f);
    const float inv = __fdiv_rn(127.0f, amax);
    uint2* tap = (live && a.xq_out && blockIdx.x == 0) ? reinterpret_cast<uint2*>(a.xq_out + static_cast<size_t>(m) * K) : nullptr;
    if (m < MT) {
      for (int i = sub * 32 + lane; i < nvec8; i += WPR * 32) {
        uint2 wd = make_uint2(0u, 0u);
        if (live) {
          const uint4 raw = xr[i];
          const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
          int q[8];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            q[2 * e] = quant_code(__uint_as_float(rw[e] << 16), inv);
            q[2 * e + 1] = quant_code(__uint_as_float(rw[e] & 0xffff0000u), inv);
          }
          wd.x = (q[0] & 0xff) | ((q[1] & 0xff) << 8) | ((q[2] & 0xff) << 16) | (static_cast<uint32_t>(q[3]) << 24);
          wd.y = (q[4] & 0xff) | ((q[5] & 0xff) << 8) | ((q[6] & 0xff) << 16) | (static_cast<uint32_t>(q[7]) << 24);
        }
        dst[i] = wd;
        if (tap) tap[i] = wd;
      }
      if (sub == 0 && lane == 0) {
        sc_s[m] = live ? __fdiv_rn(amax, 127.0f) : 0.0f;
        if (live && a.absmax_out && blockIdx.x == 0) a.absmax_out[m] = amax;
      }
    }
  }
  __syncthreads();

  const float wscale = *a.scale;
  for (int n0 = n_first; n0 < a.N; n0 += gridDim.x * (GV8_THREADS / 32) * R) {
    const uint4* wr = reinterpret_cast<const uint4*>(a.wq + static_cast<size_t>(n0) * K);
    int acc[R][MT];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int m = 0; m < MT; ++m) acc[r][m] = 0;
    auto step = [&](const uint4 (&wv)[R], int i) {
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        const uint4 xv = *reinterpret_cast<const uint4*>(xq_s + m * K + 16 * i);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          acc[r][m] = dp4a_s8s8(wv[r].x, xv.x, acc[r][m]);
          acc[r][m] = dp4a_s8s8(wv[r].y, xv.y, acc[r][m]);
          acc[r][m] = dp4a_s8s8(wv[r].z, xv.z, acc[r][m]);
          acc[r][m] = dp4a_s8s8(wv[r].w, xv.w, acc[r][m]);
        }
      }
    };
    int i = lane;
    if (n0 == n_first) {  // the steps whose weights were requested up front
#pragma unroll
      for (int p = 0; p < PRE; ++p, i += 32)
        if (i < nvec16) step(pre[p], i);
    }
#pragma unroll 2
    for (; i < nvec16; i += 32) {
      uint4 wv[R];
#pragma unroll
      for (int r = 0; r < R; ++r) wv[r] = wr[static_cast<size_t>(r) * nvec16 + i];
      step(wv, i);
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int m = 0; m < MT; ++m) acc[r][m] = warp_sum_i(acc[r][m]);
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          if (m < a.M) {
            const float yv = __fmul_rn(static_cast<float>(acc[r][m]), __fmul_rn(wscale, sc_s[m]));
            const size_t o = static_cast<size_t>(m) * a.N + n0 + r;
            if (a.acc_out) a.acc_out[o] = acc[r][m];
            if (a.out_dtype == BITRL_OUT_F32) static_cast<float*>(a.y)[o] = yv;
            else static_cast<unsigned short*>(a.y)[o] = float_to_bf16_bits(yv);
          }
        }
    }
  }
}

template <int MT, int R>
bitrl_status launch_gemv_w8_tr(const Gemv8Args& a, cudaStream_t st) {
  const size_t smem = static_cast<size_t>(MT) * a.K + MT * sizeof(float) + 16;
  BITRL_CUDA(cudaFuncSetAttribute(gemv_w8_kernel<MT, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  int grid = sm_count() * (smem <= 100 * 1024 ? 2 : 1);
  const int rows_per_cta = (GV8_THREADS / 32) * R;
  const int row_groups = (a.N + rows_per_cta - 1) / rows_per_cta;
  if (grid > row_groups) grid = row_groups;
  BITRL_CUDA(launch_pdl(gemv_w8_kernel<MT, R>, dim3(grid), dim3(GV8_THREADS), smem, st, a));
  count_launch(1);
  return BITRL_OK;
}

template <int MT>
bitrl_status launch_gemv_w8_t(const Gemv8Args& a, cudaStream_t st) {
  // Four rows per warp (two for the wide token counts).  For one or two tokens fewer rows per warp when four would leave
  // SMs without a CTA (N = 2560: 80 CTAs of 32 rows; 6912 -> 2560 at M = 1: 14.6 -> 11.6 us); from four tokens on the
  // activation reads from shared memory that fewer rows share cost more than the idle SMs (M = 4: 14.9 -> 15.6 us).
  constexpr int RMAX = MT <= 4 ? 4 : 2;
  if constexpr (MT <= 2) {
    const int ctas_wanted = sm_count();
    if (a.N / ((GV8_THREADS / 32) * 4) >= ctas_wanted) return launch_gemv_w8_tr<MT, 4>(a, st);
    if (a.N / ((GV8_THREADS / 32) * 2) >= ctas_wanted) return launch_gemv_w8_tr<MT, 2>(a, st);
    return launch_gemv_w8_tr<MT, 1>(a, st);
  } else {
    return launch_gemv_w8_tr<MT, RMAX>(a, st);
  }
}

inline bool gemv_w8_fits(int M, int K) { return M <= BITRL_GEMV_MAX_M && static_cast<size_t>(16) * K <= 200 * 1024; }

bitrl_status launch_gemv_w8(const int8_t* wq, const float* scale, int N, int K, const void* x, int M, void* y, int out_dtype,
                            int8_t* xq_out, float* absmax_out, int32_t* acc_out, cudaStream_t st) {
  Gemv8Args a{wq, scale, static_cast<const unsigned short*>(x), M, N, K, y, out_dtype, xq_out, absmax_out, acc_out};
  if (M == 1) return launch_gemv_w8_t<1>(a, st);
  if (M == 2) return launch_gemv_w8_t<2>(a, st);
  if (M <= 4) return launch_gemv_w8_t<4>(a, st);
  if (M <= 8) return launch_gemv_w8_t<8>(a, st);
  return launch_gemv_w8_t<16>(a, st);
}

// Symmetric absmax quantization of a weight matrix: pass 1 = largest magnitude (integer atomicMax on the bit pattern of a
// non-negative float: order-free, deterministic), pass 2 = codes.
__global__ void w8_absmax_kernel(const float4* W, long long n4, unsigned int* amax_bits) {
  float m = 0.0f;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n4;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const float4 v = W[i];
    m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
  }
  m = warp_max(m);
  if ((threadIdx.x & 31) == 0) atomicMax(amax_bits, __float_as_uint(m));
}
__global__ void w8_quantize_kernel(const float4* W, long long n4, const unsigned int* amax_bits, uint32_t* Wq, float* scale) {
  const float a = fmaxf(__uint_as_float(*amax_bits), 1e-20f);
  const float inv = __fdiv_rn(127.0f, a);
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n4;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const float4 v = W[i];
    const int q0 = quant_code(v.x, inv), q1 = quant_code(v.y, inv), q2 = quant_code(v.z, inv), q3 = quant_code(v.w, inv);
    Wq[i] = (q0 & 0xff) | ((q1 & 0xff) << 8) | ((q2 & 0xff) << 16) | (static_cast<uint32_t>(q3) << 24);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *scale = __fdiv_rn(a, 127.0f);
}

// amax_bits: 4 bytes of scratch inside the caller's `scale` buffer would alias the result, so the launcher uses the
// second float of a two-float scale buffer: scale[0] = result, scale[1] = scratch.
bitrl_status launch_w8_quantize(const float* W, int N, int K, int8_t* Wq, float* scale2, cudaStream_t st) {
  const long long n4 = static_cast<long long>(N) * K / 4;
  unsigned int* amax_bits = reinterpret_cast<unsigned int*>(scale2 + 1);
  BITRL_CUDA(cudaMemsetAsync(amax_bits, 0, 4, st));
  const int grid = sm_count() * 8;
  w8_absmax_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const float4*>(W), n4, amax_bits);
  w8_quantize_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const float4*>(W), n4, amax_bits,
                                           reinterpret_cast<uint32_t*>(Wq), scale2);
  count_launch(2);
  BITRL_CUDA(cudaGetLastError());
  return BITRL_OK;
}

// y = W8A8(x_q): wq dev int8 [N,K] row-major, scale dev [1], x_q dev int8 [M,K], absmax dev [M].
bitrl_status launch_gemm_w8(const int8_t* wq, const float* scale, int N, int K, const int8_t* xq, const float* absmax, int M,
                            void* y, int out_dtype, const void* residual, int32_t* acc_out, cudaStream_t st) {
  encode_tiled_fn encode = get_encode_tiled();
  if (!encode) return cuda_fail(cudaErrorSymbolNotFound);
  const int sms = sm_count();
  const int tiles_n = N / 128;
  int tok = 256, splits = 1;
  const int kblocks = K / 128;
  {
    long long best = -1;
    const int cand[5] = {256, 224, 192, 128, 64};
    for (int i = 0; i < 5; ++i) {
      const long long tiles = static_cast<long long>(tiles_n) * ((M + cand[i] - 1) / cand[i]);
      const long long waves = (tiles + sms - 1) / sms;
      const long long cost = waves * (2 * cand[i] > 300 ? 2 * cand[i] : 300);  // tensor time per k block, floor for small tiles
      if (best < 0 || cost <= best) { best = cost; tok = cand[i]; }
    }
    // Few tiles and a long K: k ranges over the CTAs of a cluster, as in the ternary GEMM (same cost model, in ns:
    // 0.9 ns per unit of the cost above; a wave of clusters pays 2 + 0.15 S + 0.015 tiles us on top of its k blocks:
    // at M = 64, 2560 -> 6912, two k ranges measured 10.9 us against 9.6 us unsplit, so the fixed part is larger here).
    if (gemm_clsk_mode() != 0) {
      long long best_ns = best * kblocks * 9 / 10;
      for (int i = 3; i < 5; ++i) {
        const long long tiles = static_cast<long long>(tiles_n) * ((M + cand[i] - 1) / cand[i]);
        if (tiles * 2 > sms) continue;
        for (int sp = 2; sp <= 8 && sp <= kblocks; ++sp) {
          const int kps = (kblocks + sp - 1) / sp;
          if ((kblocks + kps - 1) / kps != sp || !clsk_fits(cand[i], sp)) continue;
          const int clusters = gemm_w8_clsk_max_clusters(cand[i], sp);
          if (clusters <= 0) continue;
          long long cost = ((tiles + clusters - 1) / clusters) * (kps * 270LL + 2000 + 150 * sp + 15 * tiles);
          if (gemm_clsk_mode() == sp) cost = 0;  // forced size (tuning knob)
          if (cost <= best_ns) { best_ns = cost; tok = cand[i]; splits = sp; }
        }
      }
    }
  }
  // Paired CTAs for large launches (same knob as the ternary GEMM): widest tile that fills whole waves of clusters.
  bool pair = false;
  int pair_clusters = 0;
  if (gemm_pair_mode() != 0 && tiles_n % 2 == 0 && M >= G8_PAIR_MIN_M && splits == 1) {
    long long best = -1;
    int ptok = 0;
    const int cand[3] = {256, 192, 128};
    for (int i = 0; i < 3; ++i) {
      const int clusters = gemm_w8_pair_max_clusters(cand[i]);
      if (clusters <= 0) continue;
      const long long tiles = static_cast<long long>(tiles_n / 2) * ((M + cand[i] - 1) / cand[i]);
      const long long cost = ((tiles + clusters - 1) / clusters) * (2 * cand[i] > 300 ? 2 * cand[i] : 300);
      if (best < 0 || cost < best) { best = cost; ptok = cand[i]; }
    }
    if (const int forced = gemm_forced_tok())
      if (forced == 256 || forced == 192 || forced == 128) ptok = forced;
    if (ptok) {
      pair_clusters = gemm_w8_pair_max_clusters(ptok);
      if (pair_clusters > 0) { pair = true; tok = ptok; }
    }
  }
  CUtensorMap tmx, tmw;
  const cuuint32_t estr[2] = {1, 1};
  {
    const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(M)};
    const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(K)};
    const cuuint32_t box[2] = {128, static_cast<cuuint32_t>(pair ? tok / 2 : tok)};
    if (encode(&tmx, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(xq), gdim, gstride, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  {
    const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(N)};
    const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(K)};
    const cuuint32_t box[2] = {128, 128};
    if (encode(&tmw, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(wq), gdim, gstride, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cuda_fail(cudaErrorInvalidValue);
  }
  Gemm8Args a{scale, absmax, M, N, K, y, out_dtype, static_cast<const unsigned short*>(residual), acc_out, tiles_n, 0,
              splits, (kblocks + splits - 1) / splits};
  if (splits > 1) {
    a.tiles_total = tiles_n * ((M + tok - 1) / tok);
    void (*ck)(const CUtensorMap, const CUtensorMap, const Gemm8Args) = gemm_w8_clsk_kernel(tok);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(a.tiles_total * splits));  // cluster c = tile c, rank = k range
    cfg.blockDim = dim3(G8_THREADS);
    cfg.dynamicSmemBytes = G8_SMEM_BYTES;
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
    BITRL_CUDA(cudaFuncSetAttribute(ck, cudaFuncAttributeMaxDynamicSharedMemorySize, G8_SMEM_BYTES));
    BITRL_CUDA(cudaLaunchKernelEx(&cfg, ck, tmx, tmw, a));
    count_launch(1);
    return BITRL_OK;
  }
  if (pair) {
    a.tiles_n = tiles_n / 2;
    a.tiles_total = a.tiles_n * ((M + tok - 1) / tok);
    const int clusters = a.tiles_total < pair_clusters ? a.tiles_total : pair_clusters;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * clusters);
    cfg.blockDim = dim3(G8_THREADS);
    cfg.dynamicSmemBytes = G8_SMEM_BYTES;
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
    BITRL_CUDA(cudaLaunchKernelEx(&cfg, gemm_w8_pair_kernel(tok), tmx, tmw, a));
    count_launch(1);
    return BITRL_OK;
  }
  a.tiles_total = tiles_n * ((M + tok - 1) / tok);
  const int grid = a.tiles_total < sms ? a.tiles_total : sms;
  void (*kern)(const CUtensorMap, const CUtensorMap, const Gemm8Args) =
      tok == 256 ? gemm_w8_kernel<256> : tok == 224 ? gemm_w8_kernel<224> : tok == 192 ? gemm_w8_kernel<192>
      : tok == 128 ? gemm_w8_kernel<128> : gemm_w8_kernel<64>;
  BITRL_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, G8_SMEM_BYTES));
  BITRL_CUDA(launch_pdl(kern, dim3(grid), dim3(G8_THREADS), G8_SMEM_BYTES, st, tmx, tmw, a));
  count_launch(1);
  return BITRL_OK;
}

}  // namespace bitrl
