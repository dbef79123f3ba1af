// Grouped streaming kernel of the W8A8 and W4A8 layers (the higher-precision critics of Table IV): several independent
// layers with M <= 2 tokens in ONE launch, the int8 (or packed int4) weights read once at HBM speed.
//
// A single decode-size launch of this layer (35 MB at most) spends a third of its time ramping up and quantizing the
// activations; a critic backbone evaluated for one state per step is a sweep over many such matrices.  As in the
// ternary path the sweep is one persistent kernel: one CTA per SM, a producer thread that streams the row-major weights
// in slots of R whole rows (R * K <= 32 KB, one bulk copy and one mbarrier per slot) through a ring of six slots, and
// sixteen consumer warps.  A warp owns whole rows (global row index mod 16), its lanes walk a row in 16-byte steps
// (conflict-free in shared memory) and feed dp4a; one shuffle tree per row.  int8 weights are used as they are
// (signed x signed); int4 weights are two biased codes (q + 8) per byte, split into their nibble planes by two masks
// (the high plane stays at its bit position and is scaled back by an exact shift once per row) and multiplied as
// unsigned bytes with activations stored as an even-k and an odd-k plane, the bias repaid as 8 * sum_k x_q; at one token
// a warp takes two of the (half as long) int4 rows at a time, one per half-warp.  The work
// list is every job's rows in slot units, split into contiguous byte-balanced ranges, two per CTA.
#pragma once

#include <algorithm>
#include <vector>

#include "common.cuh"
#include "gemm_w8.cuh"
#include "gemv_multi.cuh"
#include "w4.cuh"
#include "ptx.cuh"

namespace bitrl {

constexpr int GV8M_CONSUMERS = 16;
constexpr int GV8M_THREADS = (GV8M_CONSUMERS + 1) * 32;
constexpr int GV8M_SLOT_BYTES = 32 * 1024;
constexpr int GV8M_DEPTH = 6;
enum { GV8M_WAIT_EMPTY = 51, GV8M_WAIT_FULL = 52 };

struct Gv8Job {
  const int8_t* wq;
  const float* scale;
  const unsigned short* x;
  void* y;
  int N, K;
  int row_bytes;      // K for int8 weights, K / 2 for packed int4
  int rows_per_slot;  // R = floor(32 KB / row_bytes), at least 1
  int unit_begin;     // index of this job's first slot unit in the global work list
};

struct Gv8mArgs {
  Gv8Job jobs[GVM_MAX_JOBS];
  int seg[GVM_MAX_CTAS][4];
  int njobs, M, out_dtype, kmax;
};

template <int MT, bool W4>
__global__ void __launch_bounds__(GV8M_THREADS, 1) gemv8_multi_kernel(const __grid_constant__ Gv8mArgs a) {
  extern __shared__ __align__(128) unsigned char gv8m_smem[];
  const uint32_t ring = ptx::smem_u32(gv8m_smem);
  int8_t* xq_s = reinterpret_cast<int8_t*>(gv8m_smem + GV8M_DEPTH * GV8M_SLOT_BYTES);  // [MT][K]
  unsigned char* tail = gv8m_smem + GV8M_DEPTH * GV8M_SLOT_BYTES + static_cast<size_t>(MT) * a.kmax;
  const uint32_t bar_full = ptx::smem_u32(tail);           // [DEPTH]
  const uint32_t bar_empty = bar_full + 8 * GV8M_DEPTH;    // [DEPTH]
  float* sc_s = reinterpret_cast<float*>(tail + 16 * GV8M_DEPTH);  // [MT] a_m / 127
  float* redf = sc_s + MT;                                         // [CONSUMERS]
  int* redi = reinterpret_cast<int*>(redf + GV8M_CONSUMERS);       // [CONSUMERS]
  int* rs_s = redi + GV8M_CONSUMERS;                               // [MT] sum_k x_q (int4 weights only)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int u_begin = a.seg[blockIdx.x][0], u_mid = a.seg[blockIdx.x][1], u_resume = a.seg[blockIdx.x][2],
            u_end = a.seg[blockIdx.x][3];

  if (threadIdx.x == 0) {
    for (int s = 0; s < GV8M_DEPTH; ++s) {
      ptx::mbar_init(bar_full + 8 * s, 1);
      ptx::mbar_init(bar_empty + 8 * s, GV8M_CONSUMERS);
    }
    ptx::mbar_init_fence();
  }
  __syncthreads();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == GV8M_CONSUMERS) {
    // ------------------------------------------------------------------ producer (weights are immutable: no wait)
    if (lane == 0) {
      uint32_t s = 0, ph = 0;
      int j = 0;
      bool ok = true;
      for (int u = u_begin == u_mid ? u_resume : u_begin; ok && u < u_end; u = (u + 1 == u_mid) ? u_resume : u + 1) {
        while (j + 1 < a.njobs && a.jobs[j + 1].unit_begin <= u) ++j;
        const Gv8Job& job = a.jobs[j];
        const int row0 = (u - job.unit_begin) * job.rows_per_slot;
        const int rows = min(job.rows_per_slot, job.N - row0);
        const uint32_t bytes = static_cast<uint32_t>(rows) * job.row_bytes;
        if (!ptx::mbar_wait(bar_empty + 8 * s, ph ^ 1u)) { report_timeout(GV8M_WAIT_EMPTY); ok = false; break; }
        ptx::mbar_arrive_expect_tx(bar_full + 8 * s, bytes);
        ptx::bulk_g2s(ring + s * GV8M_SLOT_BYTES, job.wq + static_cast<size_t>(row0) * job.row_bytes, bytes, bar_full + 8 * s);
        if (++s == GV8M_DEPTH) { s = 0; ph ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    asm volatile("griddepcontrol.wait;" ::: "memory");  // x may be produced by the preceding kernel
    const unsigned short* cached_x = nullptr;
    int cached_k = 0;
    uint32_t s = 0, ph = 0;
    int j = 0;
    bool ok = true;
    for (int u = u_begin == u_mid ? u_resume : u_begin; u < u_end; u = (u + 1 == u_mid) ? u_resume : u + 1) {
      while (j + 1 < a.njobs && a.jobs[j + 1].unit_begin <= u) ++j;
      const Gv8Job& job = a.jobs[j];
      const int K = job.K;
      if (job.x != cached_x || K != cached_k) {
        // ---- quantize this job's activations (all consumer warps per token) ----
        asm volatile("bar.sync 2, %0;" ::"n"(GV8M_CONSUMERS * 32) : "memory");
        const int nvec8 = K >> 3;
        constexpr int NTH = GV8M_CONSUMERS * 32;
        for (int m = 0; m < MT; ++m) {
          uint2* dst = reinterpret_cast<uint2*>(xq_s + m * K);
          if (m >= a.M) {
            for (int i = threadIdx.x; i < nvec8; i += NTH) dst[i] = make_uint2(0u, 0u);
            if (threadIdx.x == 0) { sc_s[m] = 0.0f; rs_s[m] = 0; }
            continue;
          }
          const uint4* xr = reinterpret_cast<const uint4*>(job.x + static_cast<size_t>(m) * K);
          float mx = 0.0f;
          for (int i = threadIdx.x; i < nvec8; i += NTH) mx = fmaxf(mx, absmax8(xr[i]));
          mx = warp_max(mx);
          if (lane == 0) redf[warp] = mx;
          asm volatile("bar.sync 2, %0;" ::"n"(GV8M_CONSUMERS * 32) : "memory");
#pragma unroll
          for (int i = 0; i < GV8M_CONSUMERS; ++i) mx = fmaxf(mx, redf[i]);
          const float amax = fmaxf(mx, 1e-5f);
          const float inv = __fdiv_rn(127.0f, amax);
          int rs = 0;
          for (int i = threadIdx.x; i < nvec8; i += NTH) {
            const uint4 raw = xr[i];
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
            if (W4) {
              // The even k and the odd k of every eight, the order the two nibble planes of a weight word come out in, go
              // to two planes of K/2 bytes each: a lane then reads 16 contiguous bytes of either plane per step and the
              // lanes of a warp read consecutive 16-byte pieces (one plane with both halves side by side made every
              // activation load a two-way bank conflict).
              rs += q[0] + q[1] + q[2] + q[3] + q[4] + q[5] + q[6] + q[7];
              uint32_t* plane = reinterpret_cast<uint32_t*>(xq_s + m * K);
              plane[i] = __byte_perm(wd.x, wd.y, 0x6420);
              plane[(K >> 3) + i] = __byte_perm(wd.x, wd.y, 0x7531);
            } else {
              dst[i] = wd;
            }
          }
          if (W4) {
            rs = warp_sum_i(rs);
            if (lane == 0) redi[warp] = rs;
          }
          asm volatile("bar.sync 2, %0;" ::"n"(GV8M_CONSUMERS * 32) : "memory");  // redf is reused by the next token
          if (threadIdx.x == 0) {
            sc_s[m] = __fdiv_rn(amax, 127.0f);
            int t = 0;
            if (W4) {
#pragma unroll
              for (int i = 0; i < GV8M_CONSUMERS; ++i) t += redi[i];
            }
            rs_s[m] = t;
          }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(GV8M_CONSUMERS * 32) : "memory");
        cached_x = job.x;
        cached_k = K;
      }

      // ---- one slot: rows row0 .. row0 + rows - 1 of the job; this warp takes those with (row mod 16) == warp ----
      const int row0 = (u - job.unit_begin) * job.rows_per_slot;
      const int rows = min(job.rows_per_slot, job.N - row0);
      const float wscale = *job.scale;
      if (ok && !ptx::mbar_wait(bar_full + 8 * s, ph)) { report_timeout(GV8M_WAIT_FULL); ok = false; }
      if (ok) {
        const int nvec16 = job.row_bytes >> 4;  // 16-byte pieces of a row: 16 int8 or 32 int4 weights each
        if constexpr (W4 && MT == 1) {
          // int4 rows are half as long, so the reduction and the epilogue of a row weigh twice as much: a warp takes
          // two rows at a time, one per half-warp (16 lanes walk a row; one four-step shuffle tree serves both rows).
          const int hl = lane & 15, hr = lane >> 4;
          for (int r2 = ((warp - (row0 >> 1)) & (GV8M_CONSUMERS - 1)) * 2; r2 < rows; r2 += 2 * GV8M_CONSUMERS) {
            const int r = r2 + hr;
            const bool live = r < rows;
            const uint32_t wrow = ring + s * GV8M_SLOT_BYTES + static_cast<uint32_t>(live ? r : r2) * job.row_bytes;
            int acc = 0, acc_hi = 0;
#pragma unroll 5
            for (int i = hl; i < nvec16; i += 16) {
              const uint4 wv = ptx::lds128(wrow + 16 * i);
              const uint4 xa = *reinterpret_cast<const uint4*>(xq_s + 16 * i);
              const uint4 xb = *reinterpret_cast<const uint4*>(xq_s + (K >> 1) + 16 * i);
              const uint32_t xe[4] = {xa.x, xa.y, xa.z, xa.w}, xo[4] = {xb.x, xb.y, xb.z, xb.w};
              const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
              for (int p = 0; p < 4; ++p) {
                acc = dp4a_u8s8(ww[p] & 0x0f0f0f0fu, static_cast<int>(xe[p]), acc);
                acc_hi = dp4a_u8s8(ww[p] & 0xf0f0f0f0u, static_cast<int>(xo[p]), acc_hi);
              }
            }
            acc += acc_hi >> 4;  // exact: a multiple of 16
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (hl == 0 && live) {
              acc -= 8 * rs_s[0];
              const float yv = __fmul_rn(static_cast<float>(acc), __fmul_rn(wscale, sc_s[0]));
              const size_t o = static_cast<size_t>(row0 + r);
              if (a.out_dtype == BITRL_OUT_F32) static_cast<float*>(job.y)[o] = yv;
              else static_cast<unsigned short*>(job.y)[o] = float_to_bf16_bits(yv);
            }
          }
        } else
        for (int r = (warp - row0) & (GV8M_CONSUMERS - 1); r < rows; r += GV8M_CONSUMERS) {
          const uint32_t wrow = ring + s * GV8M_SLOT_BYTES + static_cast<uint32_t>(r) * job.row_bytes;
          int acc[MT], acc_hi[MT];  // acc_hi: the high-nibble plane left at its bit position, i.e. 16 times its share
#pragma unroll
          for (int m = 0; m < MT; ++m) acc[m] = acc_hi[m] = 0;
#pragma unroll 4
          for (int i = lane; i < nvec16; i += 32) {
            const uint4 wv = ptx::lds128(wrow + 16 * i);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
              if (W4) {
                // word p of the piece holds k = 32 i + 8 p .. + 7; its activations are word 4 i + p of the even-k plane
                // and of the odd-k plane
                const uint4 xa = *reinterpret_cast<const uint4*>(xq_s + m * K + 16 * i);
                const uint4 xb = *reinterpret_cast<const uint4*>(xq_s + m * K + (K >> 1) + 16 * i);
                const uint32_t xe[4] = {xa.x, xa.y, xa.z, xa.w}, xo[4] = {xb.x, xb.y, xb.z, xb.w};
                const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                  acc[m] = dp4a_u8s8(ww[p] & 0x0f0f0f0fu, static_cast<int>(xe[p]), acc[m]);
                  acc_hi[m] = dp4a_u8s8(ww[p] & 0xf0f0f0f0u, static_cast<int>(xo[p]), acc_hi[m]);
                }
              } else {
                const uint4 xv = *reinterpret_cast<const uint4*>(xq_s + m * K + 16 * i);
                acc[m] = dp4a_s8s8(wv.x, xv.x, acc[m]);
                acc[m] = dp4a_s8s8(wv.y, xv.y, acc[m]);
                acc[m] = dp4a_s8s8(wv.z, xv.z, acc[m]);
                acc[m] = dp4a_s8s8(wv.w, xv.w, acc[m]);
              }
            }
          }
#pragma unroll
          for (int m = 0; m < MT; ++m) acc[m] = warp_sum_i(acc[m] + (acc_hi[m] >> 4));  // exact: a multiple of 16
          if (lane == 0) {
#pragma unroll
            for (int m = 0; m < MT; ++m) {
              if (m < a.M) {
                if (W4) acc[m] -= 8 * rs_s[m];
                const float yv = __fmul_rn(static_cast<float>(acc[m]), __fmul_rn(wscale, sc_s[m]));
                const size_t o = static_cast<size_t>(m) * job.N + row0 + r;
                if (a.out_dtype == BITRL_OUT_F32) static_cast<float*>(job.y)[o] = yv;
                else static_cast<unsigned short*>(job.y)[o] = float_to_bf16_bits(yv);
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar_empty + 8 * s);
      }
      if (++s == GV8M_DEPTH) { s = 0; ph ^= 1u; }
    }
  }
}

struct W8Matrix {
  const int8_t* wq;   // int8 [N,K], or packed int4 [N,K/2] (as bytes)
  const float* scale;
  int32_t N, K;
};

inline bool gemv8_multi_fits(int M, int kmax) {
  return M <= 2 && static_cast<size_t>(GV8M_DEPTH) * GV8M_SLOT_BYTES + static_cast<size_t>(M) * kmax + 1024 <= GVM_SMEM_BUDGET &&
         kmax <= GV8M_SLOT_BYTES;
}

template <int MT, bool W4>
bitrl_status launch_gemv8_multi_t(const Gv8mArgs& a, int grid, size_t smem, cudaStream_t st) {
  BITRL_CUDA(cudaFuncSetAttribute(gemv8_multi_kernel<MT, W4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(smem)));
  BITRL_CUDA(launch_pdl(gemv8_multi_kernel<MT, W4>, dim3(grid), dim3(GV8M_THREADS), smem, st, a));
  count_launch(1);
  return BITRL_OK;
}

// int4 = false: w[i].wq is int8 [N,K]; true: packed int4 [N,K/2].
bitrl_status launch_gemv8_multi(int count, const W8Matrix* w, const void* const* x, void* const* y, int M, int out_dtype,
                                bool int4, cudaStream_t st) {
  static thread_local Gv8mArgs a;
  int kmax = 0, units = 0;
  long long pieces = 0;  // in 1 KB, for the byte balance
  int order[GVM_MAX_JOBS];
  for (int j = 0; j < count; ++j) order[j] = j;
  std::stable_sort(order, order + count, [&](int p, int q) { return w[p].K > w[q].K; });
  static thread_local std::vector<int> sz;
  sz.clear();
  for (int i = 0; i < count; ++i) {
    const W8Matrix& m = w[order[i]];
    const int row_bytes = int4 ? m.K / 2 : m.K;
    const int R = std::max(1, GV8M_SLOT_BYTES / row_bytes);
    a.jobs[i] = Gv8Job{m.wq, m.scale, static_cast<const unsigned short*>(x[order[i]]), y[order[i]], m.N, m.K, row_bytes, R,
                       units};
    const int nslots = (m.N + R - 1) / R;
    for (int u = 0; u < nslots; ++u) {
      const int rows = std::min(R, m.N - u * R);
      const int kb = (rows * row_bytes + 1023) / 1024;
      sz.push_back(kb);
      pieces += kb;
    }
    units += nslots;
    kmax = std::max(kmax, static_cast<int>(m.K));
  }
  if (!gemv8_multi_fits(M, kmax)) return BITRL_ERR_SHAPE;
  int grid = sm_count();
  if (grid > GVM_MAX_CTAS) grid = GVM_MAX_CTAS;
  if (grid > units) grid = units;
  gvm_partition(sz, pieces, grid, a.seg);
  a.njobs = count;
  a.M = M;
  a.out_dtype = out_dtype;
  a.kmax = kmax;
  const size_t smem = static_cast<size_t>(GV8M_DEPTH) * GV8M_SLOT_BYTES + static_cast<size_t>(M) * kmax + 1024;
  if (int4) return M == 1 ? launch_gemv8_multi_t<1, true>(a, grid, smem, st) : launch_gemv8_multi_t<2, true>(a, grid, smem, st);
  return M == 1 ? launch_gemv8_multi_t<1, false>(a, grid, smem, st) : launch_gemv8_multi_t<2, false>(a, grid, smem, st);
}

}  // namespace bitrl
