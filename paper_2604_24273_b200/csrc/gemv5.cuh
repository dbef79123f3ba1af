// The denser weight format of the streaming path: five ternary weights per byte (1.6 bits per weight), decoded
// through a lookup table, as the paper's CPU inference stack does (Sec. V: ternary products become additions and
// subtractions "with lookup tables"; Abstract: 1.58-bit weights).  Same integers as the 2-bit path, 20 % fewer bytes
// from HBM; whether the decode leaves that gain standing is what this kernel exists to measure.
//
// Canonical format (compared bytewise with the oracle): [N][ceil(K/5)] bytes, byte j of row n = sum_i c[5j+i] 3^i with
// c = W_q + 1 and positions beyond K counted as c = 1 (a zero weight).
// Kernel layout ("tile5"), made once by bitrl_linear5_create:  [N/128 row tiles][P = ceil(K/160) pieces][128 rows][32 B].
// A piece is 4 KB, as in the 2-bit layout, but covers 160 k.  Lane (2*row + half) of a warp owns 16 bytes = four 32-bit
// words = 80 k of its row.  Word jw of half h covers k0 = 160 p + 80 h + 20 jw ... k0 + 19: byte b of the word holds the
// base-3 digits d0..d3 = codes of k0 + 4b + 0..3 and d4 = code of k0 + 16 + b.  So the table entry of a byte,
//   entry = d0 | d1 << 8 | d2 << 16 | d3 << 24 | d4 << 2,
// masked with 0x03030303, is the dp4a operand for activation word (k0 + 4b ..+3) as it stands, and the four d4 of a word,
// gathered by three byte permutes, pair with activation word k0 + 16..19.  The table (243 entries) is replicated once
// per shared-memory bank (entry e of lane l at word 32 e + l), so the 32 lanes' lookups never conflict.
//
// Everything else follows the grouped 2-bit kernel for M <= 2 (gemv_multi.cuh): one persistent CTA per SM, a producer
// thread streaming 32 KB slots with bulk copies, sixteen consumer warps in two groups, two work ranges per CTA.
#pragma once

#include <algorithm>
#include <vector>

#include "common.cuh"
#include "gemv_multi.cuh"
#include "ptx.cuh"

namespace bitrl {

constexpr int T5_K = 160;             // k covered by one 4 KB piece
constexpr int T5_LUT_BYTES = 243 * 32 * 4;

struct Linear5 {
  uint8_t* tiles;  // device, tile5 layout, (N/128) * pieces * 4096 bytes
  float* gamma;    // device, [1]
  int32_t N, K, pieces;
};

struct Gv5Job {
  const uint8_t* tiles;
  const float* gamma;
  const unsigned short* x;
  void* y;
  int N, K, pieces;
  int unit_begin;
};

struct Gv5Args {
  Gv5Job jobs[GVM_MAX_JOBS];
  int seg[GVM_MAX_CTAS][4];
  int njobs, M, out_dtype, depth, kpad_max;
};

// canonical 2-bit [N][K/4] -> canonical base-3 [N][ceil(K/5)], one thread per output byte
__global__ void __launch_bounds__(256) pack5_kernel(const uint8_t* __restrict__ packed2, int N, int K,
                                                    uint8_t* __restrict__ packed5) {
  const int kb5 = (K + 4) / 5;
  const long long o = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (o >= static_cast<long long>(N) * kb5) return;
  const int j = static_cast<int>(o % kb5);
  const long long n = o / kb5;
  unsigned v = 0, p = 1;
  for (int i = 0; i < 5; ++i, p *= 3) {
    const int k = 5 * j + i;
    const unsigned c = k < K ? (packed2[n * (K / 4) + (k >> 2)] >> (2 * (k & 3))) & 3u : 1u;
    v += c * p;
  }
  packed5[o] = static_cast<uint8_t>(v);
}

// canonical base-3 [N][ceil(K/5)] -> tile5, one thread per output byte
__global__ void __launch_bounds__(256) retile5_kernel(const uint8_t* __restrict__ packed5, int N, int K, int pieces,
                                                      uint8_t* __restrict__ tiles) {
  const long long total = static_cast<long long>(N) * pieces * 32;
  const long long o = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (o >= total) return;
  const int byte_in_row = static_cast<int>(o & 31);  // 8 words x 4 bytes
  const int r = static_cast<int>((o >> 5) & (TILE_ROWS - 1));
  const long long blk = o >> 12;  // (row tile, piece)
  const int p = static_cast<int>(blk % pieces);
  const long long n = (blk / pieces) * TILE_ROWS + r;
  const int word = byte_in_row >> 2, b = byte_in_row & 3;  // word 0..7 = half * 4 + jw
  const int k0 = p * T5_K + word * 20;
  const int kb5 = (K + 4) / 5;
  auto code = [&](int k) -> unsigned {
    if (k >= K) return 1u;
    unsigned v = packed5[n * kb5 + k / 5];
    for (int i = 0; i < k % 5; ++i) v /= 3;
    return v % 3;
  };
  const unsigned v = code(k0 + 4 * b) + 3 * code(k0 + 4 * b + 1) + 9 * code(k0 + 4 * b + 2) + 27 * code(k0 + 4 * b + 3) +
                     81 * code(k0 + 16 + b);
  tiles[o] = static_cast<uint8_t>(v);
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}

template <int MT>
__global__ void __launch_bounds__(GVD_THREADS, 1) gemv5_multi_kernel(const __grid_constant__ Gv5Args a) {
  extern __shared__ __align__(128) unsigned char gv5_smem[];
  const int depth = a.depth;
  const uint32_t ring = ptx::smem_u32(gv5_smem);
  uint32_t* lut = reinterpret_cast<uint32_t*>(gv5_smem + depth * GVD_SLOT_BYTES);  // [243][32]
  int8_t* xq_s = reinterpret_cast<int8_t*>(lut) + T5_LUT_BYTES;                    // [MT][kpad_max]
  unsigned char* tail = reinterpret_cast<unsigned char*>(xq_s) + static_cast<size_t>(MT) * a.kpad_max;
  const uint32_t bar_full = ptx::smem_u32(tail);    // [depth]
  const uint32_t bar_empty = bar_full + 8 * depth;  // [depth]
  float* absmax_s = reinterpret_cast<float*>(tail + 16 * depth);  // [MT]
  int* rowsum_s = reinterpret_cast<int*>(absmax_s + MT);          // [MT]
  float* redf = reinterpret_cast<float*>(rowsum_s + MT);          // [GVD_CONSUMERS]
  int* redi = reinterpret_cast<int*>(redf + GVD_CONSUMERS);       // [GVD_CONSUMERS]
  int* comb = redi + GVD_CONSUMERS;                               // [2][8 warps][16 rows][MT]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int u_begin = a.seg[blockIdx.x][0], u_mid = a.seg[blockIdx.x][1], u_resume = a.seg[blockIdx.x][2],
            u_end = a.seg[blockIdx.x][3];

  if (threadIdx.x == 0) {
    for (int s = 0; s < depth; ++s) {
      ptx::mbar_init(bar_full + 8 * s, 1);
      ptx::mbar_init(bar_empty + 8 * s, GVD_CONSUMERS);
    }
    ptx::mbar_init_fence();
  }
  // the decode table: digits of every byte value, one copy per bank
  for (int i = threadIdx.x; i < 243 * 32; i += GVD_THREADS) {
    const unsigned e = static_cast<unsigned>(i) >> 5;
    const unsigned d0 = e % 3, d1 = (e / 3) % 3, d2 = (e / 9) % 3, d3 = (e / 27) % 3, d4 = e / 81;
    lut[i] = d0 | (d1 << 8) | (d2 << 16) | (d3 << 24) | (d4 << 2);
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
        const int pieces = a.jobs[j].pieces;
        const uint8_t* src = a.jobs[j].tiles + static_cast<size_t>(u - a.jobs[j].unit_begin) * pieces * TILE_BYTES;
        for (int kb = 0; kb < pieces; kb += GVD_PIECES) {
          const uint32_t bytes = static_cast<uint32_t>(min(GVD_PIECES, pieces - kb)) * TILE_BYTES;
          if (!ptx::mbar_wait(bar_empty + 8 * s, ph ^ 1u)) { report_timeout(GVM_WAIT_EMPTY); ok = false; break; }
          ptx::mbar_arrive_expect_tx(bar_full + 8 * s, bytes);
          ptx::bulk_g2s(ring + s * GVD_SLOT_BYTES, src + static_cast<size_t>(kb) * TILE_BYTES, bytes, bar_full + 8 * s);
          if (++s == static_cast<uint32_t>(depth)) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    asm volatile("griddepcontrol.wait;" ::: "memory");  // x may be produced by the preceding kernel
    const int half = lane & 1, grp = warp >> 3, rw = warp & 7;
    const uint32_t lut_lane = ptx::smem_u32(lut) + lane * 4;
    const unsigned short* cached_x = nullptr;
    int cached_k = 0;
    uint32_t s = 0, ph = 0, tile_no = 0;
    int j = 0;
    bool ok = true;
    for (int u = u_begin == u_mid ? u_resume : u_begin; u < u_end; u = (u + 1 == u_mid) ? u_resume : u + 1, ++tile_no) {
      while (j + 1 < a.njobs && a.jobs[j + 1].unit_begin <= u) ++j;
      const Gv5Job& job = a.jobs[j];
      const int K = job.K, pieces = job.pieces, kpad = pieces * T5_K;
      if (job.x != cached_x || K != cached_k) {
        // ---- quantize this job's activations (all consumer warps per token; zeros beyond K) ----
        asm volatile("bar.sync 2, %0;" ::"n"(GVD_CONSUMERS * 32) : "memory");
        const int nvec8 = K >> 3, nvec8_pad = kpad >> 3;
        constexpr int NTH = GVD_CONSUMERS * 32;
        for (int m = 0; m < MT; ++m) {
          uint2* dst = reinterpret_cast<uint2*>(xq_s + m * a.kpad_max);
          for (int i = nvec8 + threadIdx.x; i < nvec8_pad; i += NTH) dst[i] = make_uint2(0u, 0u);
          if (m >= a.M) {
            for (int i = threadIdx.x; i < nvec8; i += NTH) dst[i] = make_uint2(0u, 0u);
            continue;
          }
          const uint4* xr = reinterpret_cast<const uint4*>(job.x + static_cast<size_t>(m) * K);
          float mx = 0.0f;
          for (int i = threadIdx.x; i < nvec8; i += NTH) mx = fmaxf(mx, absmax8(xr[i]));
          mx = warp_max(mx);
          if (lane == 0) redf[warp] = mx;
          asm volatile("bar.sync 2, %0;" ::"n"(GVD_CONSUMERS * 32) : "memory");
#pragma unroll
          for (int i = 0; i < GVD_CONSUMERS; ++i) mx = fmaxf(mx, redf[i]);
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
            rs += q[0] + q[1] + q[2] + q[3] + q[4] + q[5] + q[6] + q[7];
            dst[i] = wd;
          }
          rs = warp_sum_i(rs);
          if (lane == 0) redi[warp] = rs;
          asm volatile("bar.sync 2, %0;" ::"n"(GVD_CONSUMERS * 32) : "memory");
          if (threadIdx.x == 0) {
            int tsum = 0;
#pragma unroll
            for (int i = 0; i < GVD_CONSUMERS; ++i) tsum += redi[i];
            rowsum_s[m] = tsum;
            absmax_s[m] = __fdiv_rn(amax, 127.0f);
          }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(GVD_CONSUMERS * 32) : "memory");
        cached_x = job.x;
        cached_k = K;
      }

      // ---- one row tile: this warp's 16 rows, pieces grp and grp + GROUPS of every slot ----
      const float gamma = *job.gamma;
      int acc[MT][2];  // [0]: digits 0..3, [1]: four times the fifth digits' share
#pragma unroll
      for (int m = 0; m < MT; ++m) acc[m][0] = acc[m][1] = 0;
      const uint32_t w_lane = ring + rw * 512 + lane * 16 + grp * TILE_BYTES;
      uint32_t x_lane = ptx::smem_u32(xq_s) + half * 80 + grp * T5_K;
      for (int kb = 0; kb < pieces; kb += GVD_PIECES, x_lane += GVD_PIECES * T5_K) {
        const int np = min(GVD_PIECES, pieces - kb) - grp;
        if (ok && !ptx::mbar_wait(bar_full + 8 * s, ph)) { report_timeout(GVM_WAIT_FULL); ok = false; }
        if (ok) {
          const uint32_t w_slot = w_lane + s * GVD_SLOT_BYTES;
          uint4 wv[GVD_PPG];
#pragma unroll
          for (int pp = 0; pp < GVD_PPG; ++pp)
            if (GVD_GROUPS * pp < np) wv[pp] = ptx::lds128(w_slot + pp * GVD_GROUPS * TILE_BYTES);
#pragma unroll
          for (int pp = 0; pp < GVD_PPG; ++pp) {
            if (GVD_GROUPS * pp < np) {
              const uint32_t wword[4] = {wv[pp].x, wv[pp].y, wv[pp].z, wv[pp].w};
              uint32_t xw[MT][20];
#pragma unroll
              for (int m = 0; m < MT; ++m)
#pragma unroll
                for (int v = 0; v < 5; ++v) {
                  const uint4 t = ptx::lds128(x_lane + m * a.kpad_max + pp * GVD_GROUPS * T5_K + 16 * v);
                  xw[m][4 * v] = t.x; xw[m][4 * v + 1] = t.y; xw[m][4 * v + 2] = t.z; xw[m][4 * v + 3] = t.w;
                }
#pragma unroll
              for (int jw = 0; jw < 4; ++jw) {
                const uint32_t w = wword[jw];
                // table word of byte value B for this lane: lut_lane + 128 B
                const uint32_t e0 = lds32(lut_lane + ((w << 7) & 0x7f80u));
                const uint32_t e1 = lds32(lut_lane + ((w >> 1) & 0x7f80u));
                const uint32_t e2 = lds32(lut_lane + ((w >> 9) & 0x7f80u));
                const uint32_t e3 = lds32(lut_lane + ((w >> 17) & 0x7f80u));
                const uint32_t q4 = prmt(prmt(e0, e1, 0x4040u), prmt(e2, e3, 0x4040u), 0x5410u) & 0x0c0c0c0cu;
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                  acc[m][0] = dp4a_u8s8(e0 & 0x03030303u, static_cast<int>(xw[m][5 * jw + 0]), acc[m][0]);
                  acc[m][0] = dp4a_u8s8(e1 & 0x03030303u, static_cast<int>(xw[m][5 * jw + 1]), acc[m][0]);
                  acc[m][0] = dp4a_u8s8(e2 & 0x03030303u, static_cast<int>(xw[m][5 * jw + 2]), acc[m][0]);
                  acc[m][0] = dp4a_u8s8(e3 & 0x03030303u, static_cast<int>(xw[m][5 * jw + 3]), acc[m][0]);
                  acc[m][1] = dp4a_u8s8(q4, static_cast<int>(xw[m][5 * jw + 4]), acc[m][1]);
                }
              }
            }
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar_empty + 8 * s);
        }
        if (++s == static_cast<uint32_t>(depth)) { s = 0; ph ^= 1u; }
      }
      // ---- combine: k halves by shuffle, the warp groups through shared memory ----
      int* cb = comb + (tile_no & 1u) * (8 * 16 * MT) + (rw * 16 + (lane >> 1)) * MT;
      int tot[MT];
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        tot[m] = acc[m][0] + (acc[m][1] >> 2);  // exact: acc[m][1] is a multiple of 4
        tot[m] += __shfl_xor_sync(0xffffffffu, tot[m], 1);
        if (grp > 0 && half == 0) cb[m] = tot[m];
      }
      asm volatile("bar.sync %0, %1;" ::"r"(4 + rw), "n"(GVD_GROUPS * 32) : "memory");
      if (grp == 0 && half == 0 && ok) {
        const int n = (u - job.unit_begin) * TILE_ROWS + rw * 16 + (lane >> 1);
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          if (m < a.M) {
            const int tv = tot[m] + cb[m] - rowsum_s[m];
            const float yv = __fmul_rn(static_cast<float>(tv), __fmul_rn(gamma, absmax_s[m]));
            const size_t o = static_cast<size_t>(m) * job.N + n;
            if (a.out_dtype == BITRL_OUT_F32) static_cast<float*>(job.y)[o] = yv;
            else static_cast<unsigned short*>(job.y)[o] = float_to_bf16_bits(yv);
          }
        }
      }
    }
  }
}

inline size_t gv5_fixed_bytes(int M, int kpad_max) {
  return static_cast<size_t>(T5_LUT_BYTES) + static_cast<size_t>(M) * kpad_max + 1024 + 2 * 8 * 16 * 2 * sizeof(int);
}

template <int MT>
bitrl_status launch_gemv5_t(const Gv5Args& a, int grid, size_t smem, cudaStream_t st) {
  BITRL_CUDA(cudaFuncSetAttribute(gemv5_multi_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(smem)));
  BITRL_CUDA(launch_pdl(gemv5_multi_kernel<MT>, dim3(grid), dim3(GVD_THREADS), smem, st, a));
  count_launch(1);
  return BITRL_OK;
}

bitrl_status launch_gemv5_multi(int count, const Linear5* const* w, const void* const* x, void* const* y, int M,
                                int out_dtype, cudaStream_t st) {
  static thread_local Gv5Args a;
  int kpad_max = 0, units = 0;
  long long pieces = 0;
  int order[GVM_MAX_JOBS];
  for (int j = 0; j < count; ++j) order[j] = j;
  std::stable_sort(order, order + count, [&](int p, int q) { return w[p]->K > w[q]->K; });
  static thread_local std::vector<int> sz;
  sz.clear();
  for (int i = 0; i < count; ++i) {
    const Linear5* l = w[order[i]];
    a.jobs[i] = Gv5Job{l->tiles, l->gamma, static_cast<const unsigned short*>(x[order[i]]), y[order[i]], l->N, l->K,
                       l->pieces, units};
    units += l->N / TILE_ROWS;
    pieces += static_cast<long long>(l->N / TILE_ROWS) * l->pieces;
    sz.insert(sz.end(), l->N / TILE_ROWS, l->pieces);
    kpad_max = std::max(kpad_max, l->pieces * T5_K);
  }
  const long long room = static_cast<long long>(GVM_SMEM_BUDGET) - static_cast<long long>(gv5_fixed_bytes(M, kpad_max));
  int depth = static_cast<int>(room / (GVD_SLOT_BYTES + 16));
  if (depth > 8) depth = 8;
  if (depth < 2) return BITRL_ERR_SHAPE;
  int grid = sm_count();
  if (grid > GVM_MAX_CTAS) grid = GVM_MAX_CTAS;
  if (grid > units) grid = units;
  gvm_partition(sz, pieces, grid, a.seg);
  a.njobs = count;
  a.M = M;
  a.out_dtype = out_dtype;
  a.depth = depth;
  a.kpad_max = kpad_max;
  const size_t smem = static_cast<size_t>(GVD_SLOT_BYTES + 16) * depth + gv5_fixed_bytes(M, kpad_max);
  return M == 1 ? launch_gemv5_t<1>(a, grid, smem, st) : launch_gemv5_t<2>(a, grid, smem, st);
}

}  // namespace bitrl
