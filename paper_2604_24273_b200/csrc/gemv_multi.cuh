// Grouped streaming kernel: several independent BitLinear calls with M <= 16 in ONE launch.
//
// A single decode-size matrix is only 2-9 MB: one launch per matrix is bound by launch and dependency latency,
// not by HBM.  When several such calls are independent (a sweep over matrices, or the heads of one layer), this
// kernel streams all of their packed weights back to back at HBM speed.
//
// One persistent CTA per SM.  The work list is the concatenation of all jobs' row-tile pairs (2 x 128 rows x all K, one
// contiguous region of the tile layout), jobs sorted by K; every CTA owns two ranges of it, balanced in bytes (see
// GvmArgs::seg).
//   warp 16     producer: bulk copies (cp.async.bulk) of four consecutive 4 KB (row tile, k block) pieces of each of the
//               unit's two row tiles into a ring of 32 KB slots - 128 to 192 KB in flight per SM, independent of the
//               activations, so it runs ahead across jobs
//   warps 0-15  consumers in two groups of 8: the work unit is a PAIR of row tiles of one job, group g owns row tile g
//               of the pair and warp w of a group rows 16w..16w+15 of it over the whole K (a ring slot holds four
//               consecutive pieces of either tile).  No two warps share an output row, so nothing is combined through
//               shared memory and no barrier joins the warps: they drift apart freely, which hides the shared-memory
//               and MMA latencies.  The 2-bit codes are masked (not shifted) straight into the A fragments of a
//               warp-level integer MMA
//               (mma.sync m16n8k32, A = unsigned codes, B = signed int8 activations of 8 tokens, int32 accumulate):
//               the same instruction count serves 1 to 8 tokens (two MMAs per k step for 9 to 16), so the kernel
//               stays memory-bound where a dp4a loop would be ALU-bound from M = 4 on.
// The activations of a job are quantized into shared memory by the consumer warps when the job's x differs from the
// cached one.  All mbarrier waits are bounded; after an expiry a warp keeps walking its work list (skipping waits and
// stores) so that the consumer-wide named barriers stay matched, and the CTA exits normally.
#pragma once

#include <algorithm>
#include <vector>

#include "common.cuh"
#include "gemv.cuh"
#include "ptx.cuh"

namespace bitrl {

constexpr int GVM_MAX_JOBS = 128;
constexpr int GVM_MAX_CTAS = 192;
constexpr int GVM_GROUPS = 2;                   // warp groups; group i takes pieces i and i + 2 of every ring slot
constexpr int GVM_CONSUMERS = 8 * GVM_GROUPS;
constexpr int GVM_THREADS = (GVM_CONSUMERS + 1) * 32;
constexpr int GVM_SMEM_BUDGET = 220 * 1024;
constexpr int GVM_PPG = 4;     // 4 KB pieces of a ring slot per warp group (= per row tile of a unit)
constexpr int GVM_UNROLL = GVM_PPG * GVM_GROUPS;  // pieces per ring slot: two bulk copies, one barrier
constexpr int GVM_SLOT_BYTES = GVM_UNROLL * TILE_BYTES;
constexpr int GVM_XPAD = 16;  // bytes added to each activation row so that the 8 token rows hit different banks

enum { GVM_WAIT_EMPTY = 21, GVM_WAIT_FULL = 22 };

struct GvmJob {
  const uint8_t* tiles;
  const float* gamma;
  const unsigned short* x;
  void* y;
  int N, K;
  int unit_begin;  // index of this job's first row tile in the global work list
  int pad;
};

struct GvmArgs {
  GvmJob jobs[GVM_MAX_JOBS];
  // Work of each CTA: two ranges of the work list, [seg[c][0], seg[c][1]) then [seg[c][2], seg[c][3]).  The jobs are
  // sorted by K, largest first, so the first range holds long row tiles and the second short ones: a CTA takes long
  // tiles while they fit its share and tops up with short ones, which balances the bytes per CTA to within half a
  // short tile (one range per CTA left the slowest CTA 5 % above the mean on the 30-block sweep).
  int seg[GVM_MAX_CTAS][4];
  int njobs, M, out_dtype, depth_log2, kmax;
};

// D(16x8, int32) += A(16x32, unsigned 8-bit, row) * B(32x8, signed 8-bit, col).
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Fragment mapping used below.  Lane (g = lane/4, t = lane%4) holds weight rows g and g+8 of its warp's 16 rows.
// A row of a piece is 8 words of 16 codes; (word >> 2s) & 0x03030303 are its codes k = 16w+4s..16w+4s+3.  The order
// in which a block's 128 k enter the MMAs is free as long as both operands agree, so lane t takes words 2t and 2t+1 of
// its rows: the lanes of a warp read disjoint 8-byte pieces (every shared-memory byte is fetched once), the shifts are
// compile-time constants, and MMA step s of a block multiplies codes k = 32t+4s.. and 32t+16+4s.. of the lane's rows
// with the activations of the same k - which are simply the lane's 32 contiguous bytes of the plain int8 row.
template <int NT>
__global__ void __launch_bounds__(GVM_THREADS, 1) gemv_multi_kernel(const __grid_constant__ GvmArgs a) {
  extern __shared__ __align__(128) unsigned char gvm_smem[];
  const int depth = 1 << a.depth_log2;
  const uint32_t ring = ptx::smem_u32(gvm_smem);
  unsigned char* xq_s = gvm_smem + depth * GVM_SLOT_BYTES;  // [NT][K + GVM_XPAD] int8 rows
  const uint32_t xq_addr = ptx::smem_u32(xq_s);
  unsigned char* tail = xq_s + static_cast<size_t>(NT) * (a.kmax + GVM_XPAD);
  const uint32_t bar_full = ptx::smem_u32(tail);    // [depth]
  const uint32_t bar_empty = bar_full + 8 * depth;  // [depth]
  float* absmax_s = reinterpret_cast<float*>(tail + 16 * depth);  // [NT] a_m / 127
  int* rowsum_s = reinterpret_cast<int*>(absmax_s + NT);          // [NT]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int u_begin = a.seg[blockIdx.x][0], u_mid = a.seg[blockIdx.x][1], u_resume = a.seg[blockIdx.x][2],
            u_end = a.seg[blockIdx.x][3];  // units u_begin..u_mid-1, then u_resume..u_end-1

  if (threadIdx.x == 0) {
    for (int s = 0; s < depth; ++s) {
      ptx::mbar_init(bar_full + 8 * s, 1);
      ptx::mbar_init(bar_empty + 8 * s, GVM_CONSUMERS);
    }
    ptx::mbar_init_fence();
  }
  __syncthreads();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == GVM_CONSUMERS) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t pc = 0;
      int j = 0;
      bool ok = true;
      for (int u = u_begin == u_mid ? u_resume : u_begin; ok && u < u_end; u = (u + 1 == u_mid) ? u_resume : u + 1) {
        while (j + 1 < a.njobs && a.jobs[j + 1].unit_begin <= u) ++j;
        const int kblocks = a.jobs[j].K / TILE_K;
        const int tile0 = 2 * (u - a.jobs[j].unit_begin);
        const int ntiles = min(2, a.jobs[j].N / TILE_ROWS - tile0);  // 1 for the half unit of an odd job
        const uint8_t* src = a.jobs[j].tiles + static_cast<size_t>(tile0) * kblocks * TILE_BYTES;
        for (int kb = 0; kb < kblocks; kb += GVM_PPG, ++pc) {
          const uint32_t bytes = static_cast<uint32_t>(min(GVM_PPG, kblocks - kb)) * TILE_BYTES;
          const uint32_t s = pc & (depth - 1), ph = (pc >> a.depth_log2) & 1u;
          if (!ptx::mbar_wait(bar_empty + 8 * s, ph ^ 1u)) { report_timeout(GVM_WAIT_EMPTY); ok = false; break; }
          ptx::mbar_arrive_expect_tx(bar_full + 8 * s, bytes * ntiles);
          for (int t = 0; t < ntiles; ++t)
            ptx::bulk_g2s(ring + s * GVM_SLOT_BYTES + t * GVM_PPG * TILE_BYTES,
                          src + (static_cast<size_t>(t) * kblocks + kb) * TILE_BYTES, bytes, bar_full + 8 * s);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    asm volatile("griddepcontrol.wait;" ::: "memory");  // x may be produced by the preceding kernel
    const int g = lane >> 2, t = lane & 3;
    const int grp = warp >> 3, rw = warp & 7;
    const unsigned short* cached_x = nullptr;
    int cached_k = 0;
    uint32_t pc = 0;
    int j = 0;
    bool ok = true;
    for (int u = u_begin == u_mid ? u_resume : u_begin; u < u_end; u = (u + 1 == u_mid) ? u_resume : u + 1) {
      while (j + 1 < a.njobs && a.jobs[j + 1].unit_begin <= u) ++j;
      const GvmJob& job = a.jobs[j];
      const int K = job.K, kblocks = K / TILE_K;
      const int xstride = K + GVM_XPAD;
      if (job.x != cached_x || K != cached_k) {
        // ---- quantize this job's activations: one warp per token, so the tokens proceed side by side with warp-local
        // reductions only (the ring keeps filling meanwhile) ----
        asm volatile("bar.sync 2, %0;" ::"n"(GVM_CONSUMERS * 32) : "memory");  // done with the previous contents
        const int nvec8 = K >> 3;
        for (int m = warp; m < NT; m += GVM_CONSUMERS) {
          unsigned char* row = xq_s + static_cast<size_t>(m) * xstride;
          if (m >= a.M) {
            for (int i = lane; i < (xstride >> 2); i += 32) reinterpret_cast<uint32_t*>(row)[i] = 0u;
            continue;
          }
          const uint4* xr = reinterpret_cast<const uint4*>(job.x + static_cast<size_t>(m) * K);
          float mx = 0.0f;
#pragma unroll 4
          for (int i = lane; i < nvec8; i += 32) mx = fmaxf(mx, absmax8(xr[i]));
          const float amax = fmaxf(warp_max(mx), 1e-5f);
          const float inv = __fdiv_rn(127.0f, amax);
          int rs = 0;
#pragma unroll 2
          for (int i = lane; i < nvec8; i += 32) {
            const uint4 raw = xr[i];
            const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
            int q[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              q[2 * e] = quant_code(__uint_as_float(rw[e] << 16), inv);
              q[2 * e + 1] = quant_code(__uint_as_float(rw[e] & 0xffff0000u), inv);
            }
            const uint32_t lo = (q[0] & 0xff) | ((q[1] & 0xff) << 8) | ((q[2] & 0xff) << 16) | (static_cast<uint32_t>(q[3]) << 24);
            const uint32_t hi = (q[4] & 0xff) | ((q[5] & 0xff) << 8) | ((q[6] & 0xff) << 16) | (static_cast<uint32_t>(q[7]) << 24);
            rs += q[0] + q[1] + q[2] + q[3] + q[4] + q[5] + q[6] + q[7];
            reinterpret_cast<uint2*>(row)[i] = make_uint2(lo, hi);
          }
          rs = warp_sum_i(rs);
          if (lane == 0) {
            rowsum_s[m] = rs;
            absmax_s[m] = __fdiv_rn(amax, 127.0f);  // the epilogue's scale is gamma * (a_m / 127)
          }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(GVM_CONSUMERS * 32) : "memory");
        cached_x = job.x;
        cached_k = K;
      }

      // ---- one unit: this warp's 16 rows of row tile `grp` of the pair, over the whole K ----
      const int tile = 2 * (u - job.unit_begin) + grp;
      const bool have_tile = tile < job.N / TILE_ROWS;  // false for group 1 in the half unit of an odd job
      const float gamma = *job.gamma;  // requested now, needed after the k loop: its latency hides behind the loop
      // The pieces of a slot are fetched from shared memory together and feed independent accumulator chains, so that
      // neither the loads nor the MMAs of one piece wait for those of another.
      constexpr int CH = NT == 8 ? 8 : 4;  // independent accumulator chains (the warp MMA has a long latency)
      int acc[CH][NT / 8][4];
#pragma unroll
      for (int c = 0; c < CH; ++c)
#pragma unroll
        for (int h = 0; h < NT / 8; ++h)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[c][h][e] = 0;
      const uint32_t xlane = xq_addr + g * xstride + t * 32;
      const uint32_t wlane = ring + grp * GVM_PPG * TILE_BYTES + rw * 512 + g * 32 + t * 8;
      for (int kb = 0; kb < kblocks; kb += GVM_PPG) {
        const int np = min(GVM_PPG, kblocks - kb);
        uint2 wr[GVM_PPG][2];
        const uint32_t s = pc & (depth - 1), ph = (pc >> a.depth_log2) & 1u;
        if (ok && !ptx::mbar_wait(bar_full + 8 * s, ph)) { report_timeout(GVM_WAIT_FULL); ok = false; }
        if (ok) {
          if (have_tile) {
#pragma unroll
            for (int p = 0; p < GVM_PPG; ++p) {
              if (p < np) {
                const uint32_t wslice = wlane + s * GVM_SLOT_BYTES + p * TILE_BYTES;
                wr[p][0] = ptx::lds64(wslice);
                wr[p][1] = ptx::lds64(wslice + 8 * 32);
              }
            }
#pragma unroll
            for (int p = 0; p < GVM_PPG; ++p) {
              if (p < np) {
#pragma unroll
                for (int h = 0; h < NT / 8; ++h) {
                  const uint32_t xa_addr = xlane + h * 8 * xstride + (kb + p) * TILE_K;
                  const uint4 xa = ptx::lds128(xa_addr), xb = ptx::lds128(xa_addr + 16);
                  const uint32_t xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
                  for (int ks = 0; ks < 4; ++ks) {
                    // The codes stay at their bit positions (c * 4^ks still fits an unsigned byte): one mask and no
                    // shift per operand.  Chain ks then holds 4^ks times its share and is scaled back once per tile.
                    const uint32_t msk = 0x03030303u << (2 * ks);
                    mma_u8s8(acc[((p * 4) % CH) + ks][h], wr[p][0].x & msk, wr[p][1].x & msk, wr[p][0].y & msk,
                             wr[p][1].y & msk, xv[ks], xv[4 + ks]);
                  }
                }
              }
            }
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar_empty + 8 * s);
        }
        ++pc;
      }
#pragma unroll
      for (int c = 1; c < CH; ++c)
#pragma unroll
        for (int h = 0; h < NT / 8; ++h)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[0][h][e] += acc[c][h][e] >> (2 * (c & 3));  // exact: multiples of 4^(c&3)
      if (have_tile && ok) {
        // C fragment: acc[h][0..1] = (row g, tokens 8h+2t, +1), acc[h][2..3] = (row g+8, same tokens)
        const int n0 = tile * TILE_ROWS + rw * 16 + g;
#pragma unroll
        for (int h = 0; h < NT / 8; ++h)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int m = 8 * h + 2 * t + (e & 1);
            if (m < a.M) {
              const int tv = acc[0][h][e] - rowsum_s[m];
              const float yv = __fmul_rn(static_cast<float>(tv), __fmul_rn(gamma, absmax_s[m]));
              const size_t o = static_cast<size_t>(m) * job.N + n0 + (e >> 1) * 8;
              if (a.out_dtype == BITRL_OUT_F32) static_cast<float*>(job.y)[o] = yv;
              else static_cast<unsigned short*>(job.y)[o] = float_to_bf16_bits(yv);
            }
          }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// M <= 2 variant: dp4a instead of the warp MMA (cheaper when only one or two tokens use the weights).
// The work unit is a PAIR of row tiles of one job (256 rows): warp group g (8 warps) owns row tile g of the pair, warp w
// of a group rows 16w..16w+15 of that tile over the whole K, lane = 2*row + k half as in the single-matrix kernel.  A
// ring slot holds four consecutive 4 KB pieces of either tile (two bulk copies, one barrier).  Since no two warps
// share an output row, nothing is combined through shared memory and no barrier joins the warps: they drift apart
// freely, which is what hides the shared-memory and dp4a latencies (two groups on the SAME rows with a pair barrier per
// tile left every warp waiting for its partner's epilogue).  A job with an odd number of row tiles ends in a half unit.
constexpr int GVD_GROUPS = 2;
constexpr int GVD_CONSUMERS = 8 * GVD_GROUPS;
constexpr int GVD_THREADS = (GVD_CONSUMERS + 1) * 32;
constexpr int GVD_PPG = 4;                                 // pieces of a slot per group (= per row tile of the pair)
constexpr int GVD_PIECES = GVD_PPG * GVD_GROUPS;           // 4 KB pieces per ring slot
constexpr int GVD_SLOT_BYTES = GVD_PIECES * TILE_BYTES;

template <int MT>
__global__ void __launch_bounds__(GVD_THREADS, 1) gemv_multi_dp4a_kernel(const __grid_constant__ GvmArgs a) {
  extern __shared__ __align__(128) unsigned char gvm_smem[];
  const int depth = a.depth_log2;  // for this kernel the field holds the number of ring slots itself
  const uint32_t ring = ptx::smem_u32(gvm_smem);
  int8_t* xq_s = reinterpret_cast<int8_t*>(gvm_smem + depth * GVD_SLOT_BYTES);  // [MT][K]
  unsigned char* tail = gvm_smem + depth * GVD_SLOT_BYTES + static_cast<size_t>(MT) * a.kmax;
  const uint32_t bar_full = ptx::smem_u32(tail);    // [depth]
  const uint32_t bar_empty = bar_full + 8 * depth;  // [depth]
  float* absmax_s = reinterpret_cast<float*>(tail + 16 * depth);  // [MT]
  int* rowsum_s = reinterpret_cast<int*>(absmax_s + MT);          // [MT]
  float* redf = reinterpret_cast<float*>(rowsum_s + MT);          // [GVD_CONSUMERS]
  int* redi = reinterpret_cast<int*>(redf + GVD_CONSUMERS);       // [GVD_CONSUMERS]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int u_begin = a.seg[blockIdx.x][0], u_mid = a.seg[blockIdx.x][1], u_resume = a.seg[blockIdx.x][2],
            u_end = a.seg[blockIdx.x][3];  // units u_begin..u_mid-1, then u_resume..u_end-1

  if (threadIdx.x == 0) {
    for (int s = 0; s < depth; ++s) {
      ptx::mbar_init(bar_full + 8 * s, 1);
      ptx::mbar_init(bar_empty + 8 * s, GVD_CONSUMERS);
    }
    ptx::mbar_init_fence();
  }
  __syncthreads();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == GVD_CONSUMERS) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t s = 0, ph = 0;
      int j = 0;
      bool ok = true;
      for (int u = u_begin == u_mid ? u_resume : u_begin; ok && u < u_end; u = (u + 1 == u_mid) ? u_resume : u + 1) {
        while (j + 1 < a.njobs && a.jobs[j + 1].unit_begin <= u) ++j;
        const int kblocks = a.jobs[j].K / TILE_K;
        const int tile0 = 2 * (u - a.jobs[j].unit_begin);
        const int ntiles = min(2, a.jobs[j].N / TILE_ROWS - tile0);  // 1 for the half unit of an odd job
        const uint8_t* src = a.jobs[j].tiles + static_cast<size_t>(tile0) * kblocks * TILE_BYTES;
        for (int kb = 0; kb < kblocks; kb += GVD_PPG) {
          const uint32_t bytes = static_cast<uint32_t>(min(GVD_PPG, kblocks - kb)) * TILE_BYTES;
          if (!ptx::mbar_wait(bar_empty + 8 * s, ph ^ 1u)) { report_timeout(GVM_WAIT_EMPTY); ok = false; break; }
          ptx::mbar_arrive_expect_tx(bar_full + 8 * s, bytes * ntiles);
          for (int t = 0; t < ntiles; ++t)
            ptx::bulk_g2s(ring + s * GVD_SLOT_BYTES + t * GVD_PPG * TILE_BYTES,
                          src + (static_cast<size_t>(t) * kblocks + kb) * TILE_BYTES, bytes, bar_full + 8 * s);
          if (++s == static_cast<uint32_t>(depth)) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    asm volatile("griddepcontrol.wait;" ::: "memory");  // x may be produced by the preceding kernel
    const int half = lane & 1, grp = warp >> 3, rw = warp & 7;
    const unsigned short* cached_x = nullptr;
    int cached_k = 0;
    uint32_t s = 0, ph = 0;
    int j = 0;
    bool ok = true;
    for (int u = u_begin == u_mid ? u_resume : u_begin; u < u_end; u = (u + 1 == u_mid) ? u_resume : u + 1) {
      while (j + 1 < a.njobs && a.jobs[j + 1].unit_begin <= u) ++j;
      const GvmJob& job = a.jobs[j];
      const int K = job.K, kblocks = K / TILE_K;
      if (job.x != cached_x || K != cached_k) {
        asm volatile("bar.sync 2, %0;" ::"n"(GVD_CONSUMERS * 32) : "memory");  // done with the previous contents
        const int nvec8 = K >> 3;
        for (int m = 0; m < MT; ++m) {
          uint2* dst = reinterpret_cast<uint2*>(xq_s + m * K);
          if (m >= a.M) {
            for (int i = threadIdx.x; i < nvec8; i += GVD_CONSUMERS * 32) dst[i] = make_uint2(0u, 0u);
            continue;
          }
          // The first two vectors of every thread (rows up to 8192 values) stay in registers between the absmax pass
          // and the quantization pass: one trip to global memory instead of two.
          const uint4* xr = reinterpret_cast<const uint4*>(job.x + static_cast<size_t>(m) * K);
          constexpr int NTH = GVD_CONSUMERS * 32;
          uint4 held[2];
#pragma unroll
          for (int jv = 0; jv < 2; ++jv) {
            const int i = threadIdx.x + jv * NTH;
            held[jv] = i < nvec8 ? xr[i] : make_uint4(0u, 0u, 0u, 0u);
          }
          float mx = fmaxf(absmax8(held[0]), absmax8(held[1]));
          for (int i = threadIdx.x + 2 * NTH; i < nvec8; i += NTH) mx = fmaxf(mx, absmax8(xr[i]));
          mx = warp_max(mx);
          if (lane == 0) redf[warp] = mx;
          asm volatile("bar.sync 2, %0;" ::"n"(GVD_CONSUMERS * 32) : "memory");
#pragma unroll
          for (int i = 0; i < GVD_CONSUMERS; ++i) mx = fmaxf(mx, redf[i]);
          const float amax = fmaxf(mx, 1e-5f);
          const float inv = __fdiv_rn(127.0f, amax);
          int rs = 0;
          auto quant8 = [&](const uint4 raw, int i) {
            const uint32_t rwd[4] = {raw.x, raw.y, raw.z, raw.w};
            int q[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              q[2 * e] = quant_code(__uint_as_float(rwd[e] << 16), inv);
              q[2 * e + 1] = quant_code(__uint_as_float(rwd[e] & 0xffff0000u), inv);
            }
            uint2 wd;
            wd.x = (q[0] & 0xff) | ((q[1] & 0xff) << 8) | ((q[2] & 0xff) << 16) | (static_cast<uint32_t>(q[3]) << 24);
            wd.y = (q[4] & 0xff) | ((q[5] & 0xff) << 8) | ((q[6] & 0xff) << 16) | (static_cast<uint32_t>(q[7]) << 24);
            rs += q[0] + q[1] + q[2] + q[3] + q[4] + q[5] + q[6] + q[7];
            dst[i] = wd;
          };
#pragma unroll
          for (int jv = 0; jv < 2; ++jv) {
            const int i = threadIdx.x + jv * NTH;
            if (i < nvec8) quant8(held[jv], i);
          }
          for (int i = threadIdx.x + 2 * NTH; i < nvec8; i += NTH) quant8(xr[i], i);
          rs = warp_sum_i(rs);
          if (lane == 0) redi[warp] = rs;
          asm volatile("bar.sync 2, %0;" ::"n"(GVD_CONSUMERS * 32) : "memory");
          if (threadIdx.x == 0) {
            int tsum = 0;
#pragma unroll
            for (int i = 0; i < GVD_CONSUMERS; ++i) tsum += redi[i];
            rowsum_s[m] = tsum;
            absmax_s[m] = __fdiv_rn(amax, 127.0f);  // the epilogue's scale is gamma * (a_m / 127)
          }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(GVD_CONSUMERS * 32) : "memory");
        cached_x = job.x;
        cached_k = K;
      }

      // ---- one unit: this warp's 16 rows of row tile `grp` of the pair, over the whole K ----
      const int tile = 2 * (u - job.unit_begin) + grp;
      const bool have_tile = tile < job.N / TILE_ROWS;  // false for group 1 in the half unit of an odd job
      const float gamma = *job.gamma;  // requested now, needed after the k loop: its latency hides behind the loop
      int acc[MT][4];
#pragma unroll
      for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[m][c] = 0;
      // All addresses below are 32-bit shared-memory addresses with compile-time offsets, so that a piece costs its
      // loads, masks and dp4a and little else.
      const uint32_t w_lane = ring + rw * 512 + lane * 16 + grp * GVD_PPG * TILE_BYTES;  // this lane's 16 bytes of a piece
      uint32_t x_lane = ptx::smem_u32(xq_s) + half * 64;                                 // its 64 activations of that piece
      for (int kb = 0; kb < kblocks; kb += GVD_PPG, x_lane += GVD_PPG * TILE_K) {
        const int np = min(GVD_PPG, kblocks - kb);
        if (ok && !ptx::mbar_wait(bar_full + 8 * s, ph)) { report_timeout(GVM_WAIT_FULL); ok = false; }
        if (ok) {
          if (have_tile) {
            const uint32_t w_slot = w_lane + s * GVD_SLOT_BYTES;
            uint4 wv[GVD_PPG];
#pragma unroll
            for (int pp = 0; pp < GVD_PPG; ++pp)
              if (pp < np) wv[pp] = ptx::lds128(w_slot + pp * TILE_BYTES);
#pragma unroll
            for (int pp = 0; pp < GVD_PPG; ++pp) {
              if (pp < np) {
                const uint32_t wword[4] = {wv[pp].x, wv[pp].y, wv[pp].z, wv[pp].w};
#pragma unroll
                for (int jw = 0; jw < 4; ++jw) {
                  // The codes are left at their bit positions (c1 * 4, c2 * 16, c3 * 64 still fit an unsigned byte):
                  // four masks and no shifts.  Accumulator i then holds 4^i times its share of the dot product and is
                  // scaled back by an exact shift once per row tile.
                  const uint32_t c0 = wword[jw] & 0x03030303u;
                  const uint32_t c1 = wword[jw] & 0x0c0c0c0cu;
                  const uint32_t c2 = wword[jw] & 0x30303030u;
                  const uint32_t c3 = wword[jw] & 0xc0c0c0c0u;
#pragma unroll
                  for (int m = 0; m < MT; ++m) {
                    const uint4 xv = ptx::lds128(x_lane + m * K + pp * TILE_K + 16 * jw);
                    acc[m][0] = dp4a_u8s8(c0, static_cast<int>(xv.x), acc[m][0]);
                    acc[m][1] = dp4a_u8s8(c1, static_cast<int>(xv.y), acc[m][1]);
                    acc[m][2] = dp4a_u8s8(c2, static_cast<int>(xv.z), acc[m][2]);
                    acc[m][3] = dp4a_u8s8(c3, static_cast<int>(xv.w), acc[m][3]);
                  }
                }
              }
            }
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar_empty + 8 * s);
        }
        if (++s == static_cast<uint32_t>(depth)) { s = 0; ph ^= 1u; }
      }
      // ---- epilogue of this warp's 16 rows: the k halves meet by one shuffle ----
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        int tot = acc[m][0] + (acc[m][1] >> 2) + (acc[m][2] >> 4) + (acc[m][3] >> 6);  // exact: multiples of 4^i
        tot += __shfl_xor_sync(0xffffffffu, tot, 1);
        if (half == 0 && have_tile && ok && m < a.M) {
          const int n = tile * TILE_ROWS + rw * 16 + (lane >> 1);
          const float yv = __fmul_rn(static_cast<float>(tot - rowsum_s[m]), __fmul_rn(gamma, absmax_s[m]));
          const size_t o = static_cast<size_t>(m) * job.N + n;
          if (a.out_dtype == BITRL_OUT_F32) static_cast<float*>(job.y)[o] = yv;
          else static_cast<unsigned short*>(job.y)[o] = float_to_bf16_bits(yv);
        }
      }
    }
  }
}

// Host side: builds the work list split and launches.  `w`, `x`, `y` are host arrays of `count` entries.
template <int NT>
bitrl_status launch_gemv_multi_t(const GvmArgs& a, int grid, size_t smem, cudaStream_t st) {
  BITRL_CUDA(cudaFuncSetAttribute(gemv_multi_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(smem)));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(GVM_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  BITRL_CUDA(cudaLaunchKernelEx(&cfg, gemv_multi_kernel<NT>, a));
  count_launch(1);
  return BITRL_OK;
}

template <int MT>
bitrl_status launch_gemv_multi_dp4a_t(const GvmArgs& a, int grid, size_t smem, cudaStream_t st) {
  BITRL_CUDA(cudaFuncSetAttribute(gemv_multi_dp4a_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(smem)));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(GVD_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  BITRL_CUDA(cudaLaunchKernelEx(&cfg, gemv_multi_dp4a_kernel<MT>, a));
  count_launch(1);
  return BITRL_OK;
}

inline int gvm_nt(int M) { return M <= 8 ? 8 : 16; }
// Shared memory beside the ring: activations (+ barriers, reduction scratch, the group-combine buffer).
inline size_t gvm_fixed_bytes(int M, int kmax) {
  if (M <= 2) return static_cast<size_t>(M) * kmax + 1024 + 2 * (GVD_GROUPS - 1) * 8 * 16 * 2 * sizeof(int);
  return static_cast<size_t>(gvm_nt(M)) * (kmax + GVM_XPAD) + 1024 + 2 * 8 * (gvm_nt(M) / 8) * 4 * 32 * sizeof(int);
}

// Ring depth (log2) that fits beside the activations, or -1.
inline int gvm_depth_log2(int M, int kmax) {
  for (int d = 3; d >= 1; --d)
    if (gvm_fixed_bytes(M, kmax) + (static_cast<size_t>(GVM_SLOT_BYTES) + 16) * (1u << d) <= GVM_SMEM_BUDGET) return d;
  return -1;
}

// Two ranges per CTA (see GvmArgs::seg): long units from the head of the work list while they fit the CTA's share of
// the remaining pieces, then short units from the tail up to the nearest fit.  `sz` = pieces of every unit in list order.
inline void gvm_partition(const std::vector<int>& sz, long long pieces, int grid, int (*seg)[4]) {
  int head = 0, tail = static_cast<int>(sz.size());
  long long remaining = pieces;
  for (int c = 0; c < grid; ++c) {
    const double target = static_cast<double>(remaining) / (grid - c);
    long long load = 0;
    seg[c][0] = head;
    while (head < tail && (c == grid - 1 || load + sz[head] <= target)) load += sz[head++];
    seg[c][1] = head;
    seg[c][3] = tail;
    while (head < tail && load + sz[tail - 1] <= target + 0.5 * sz[tail - 1]) load += sz[--tail];
    seg[c][2] = tail;
    remaining -= load;
  }
}

bitrl_status launch_gemv_multi(int count, const Linear* const* w, const void* const* x, void* const* y, int M,
                               int out_dtype, cudaStream_t st) {
  static thread_local GvmArgs a;  // 7 KB, kept off the stack
  int kmax = 0, units = 0;
  long long pieces = 0;
  int order[GVM_MAX_JOBS];  // jobs by K, largest first (stable)
  for (int j = 0; j < count; ++j) order[j] = j;
  std::stable_sort(order, order + count, [&](int x, int y) { return w[x]->K > w[y]->K; });
  const bool pairs = true;  // the unit of both kernels is a pair of row tiles (one per warp group)
  static thread_local std::vector<int> sz;  // 4 KB pieces of every unit, in work-list order
  sz.clear();
  for (int i = 0; i < count; ++i) {
    const int j = order[i];
    a.jobs[i] = GvmJob{w[j]->tiles, w[j]->gamma, static_cast<const unsigned short*>(x[j]), y[j], w[j]->N, w[j]->K,
                       units, 0};
    const int tiles = w[j]->N / TILE_ROWS, kb = w[j]->K / TILE_K;
    if (pairs) {
      sz.insert(sz.end(), tiles / 2, 2 * kb);
      if (tiles & 1) sz.push_back(kb);
      units += (tiles + 1) / 2;
    } else {
      sz.insert(sz.end(), tiles, kb);
      units += tiles;
    }
    pieces += static_cast<long long>(tiles) * kb;
    if (w[j]->K > kmax) kmax = w[j]->K;
  }
  int dlog = gvm_depth_log2(M, kmax);
  if (M <= 2) {  // the dp4a kernel takes the slot count itself (any count from 2 to 8)
    const long long room = static_cast<long long>(GVM_SMEM_BUDGET) - static_cast<long long>(gvm_fixed_bytes(M, kmax));
    dlog = static_cast<int>(room / (GVD_SLOT_BYTES + 16));
    if (dlog > 8) dlog = 8;
    if (dlog < 2) dlog = -1;
  }
  if (dlog < 0) return BITRL_ERR_SHAPE;
  int grid = sm_count();
  if (grid > GVM_MAX_CTAS) grid = GVM_MAX_CTAS;
  if (grid > units) grid = units;
  gvm_partition(sz, pieces, grid, a.seg);
  a.njobs = count;
  a.M = M;
  a.out_dtype = out_dtype;
  a.depth_log2 = dlog;
  a.kmax = kmax;
  const size_t smem = (M <= 2 ? static_cast<size_t>(GVD_SLOT_BYTES + 16) * dlog
                              : static_cast<size_t>(GVM_SLOT_BYTES + 16) * (1u << dlog)) + gvm_fixed_bytes(M, kmax);
  if (M == 1) return launch_gemv_multi_dp4a_t<1>(a, grid, smem, st);
  if (M == 2) return launch_gemv_multi_dp4a_t<2>(a, grid, smem, st);
  return gvm_nt(M) == 8 ? launch_gemv_multi_t<8>(a, grid, smem, st) : launch_gemv_multi_t<16>(a, grid, smem, st);
}

}  // namespace bitrl
