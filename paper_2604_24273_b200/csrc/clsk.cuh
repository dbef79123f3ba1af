// Split-K inside a thread-block cluster: the exchange of partial sums and the epilogue, shared by the ternary GEMM
// (gemm.cuh) and the int8-weight GEMM (gemm_w8.cuh).
//
// The S CTAs of a cluster hold, each in its own tensor memory, the int32 partial sums of ONE 128-row x TOK-token tile
// over their k ranges.  Token columns are dealt to the ranks in units of 8 (unit range [r U / S, (r+1) U / S) to rank
// r, U = units that hold tokens).  A CTA sends every peer the partial sums of that peer's columns through distributed
// shared memory, all threads of the cluster pass one barrier, then each CTA adds the S - 1 received slices to its own
// and applies the epilogue to its columns.  Integer sums: exact and independent of the order.
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace bitrl {

// Shared memory set aside for received partial sums (4 KB per unit of 8 token columns and sender).
__host__ __device__ constexpr uint32_t clsk_recv_bytes(int tok) { return tok <= 64 ? 49152u : 65536u; }

// Does a cluster of `S` CTAs fit the receive area of a `tok`-token tile?
inline bool clsk_fits(int tok, int S) {
  const int units = tok / 8;
  return S >= 2 && S <= 8 && static_cast<uint32_t>((S - 1) * ((units + S - 1) / S)) * 4096u <= clsk_recv_bytes(tok);
}

struct ClskArgs {
  uint32_t acc_tmem;    // tensor-memory address of this CTA's accumulator (lane 0, first token column)
  uint32_t recv_base;   // shared::cta address of the receive area (same offset in every CTA of the cluster)
  uint32_t sc_addr;     // shared::cta address of TOK floats: per-token output scale (staged here)
  uint32_t rs_addr;     // shared::cta address of TOK int32: per-token row-sum correction (staged here)
  uint32_t rank;        // this CTA's rank in the cluster
  int S;                // cluster size = k ranges per tile
  int tn, tm;           // tile coordinates: weight rows [128 tn, +128), tokens [TOK tm, +TOK)
  int M, N;
  float mul;            // gamma (ternary) or the weight scale (int8): scale_m = out_scale(mul, absmax[m])
  const float* absmax;  // [M]
  const int32_t* rowsum;  // [M] or nullptr (no correction)
  void* y;
  int out_dtype;
  const unsigned short* residual;  // nullptr or bf16 [M,N]
  int32_t* acc_out;                // nullptr or int32 [M,N]
  const volatile uint32_t* failed;  // the CTA's failure word (polled after the barrier)
};

// Called by the four epilogue warps (128 threads, named barrier 1) of every CTA of the cluster.  `q` = tensor-memory
// lane quarter of the calling warp, `ep` = 0..127 index among the epilogue threads.  `wait_acc()` waits (bounded) for
// this CTA's accumulator and returns false on a time-out.  Every calling thread passes exactly one cluster barrier,
// whatever happens.  Returns false when the accumulator wait failed (the caller reports it).
template <int TOK, class WaitAcc>
__device__ __forceinline__ bool clsk_exchange_epilogue(const ClskArgs& c, int q, int lane, int ep, WaitAcc wait_acc) {
  // These warps are idle during the main loop, so everything the epilogue reads from global memory is requested
  // first: the per-token scales and row sums go to shared memory, the residual values of the first unit of this CTA's
  // columns to registers (the later units' are requested one unit ahead).  Loading them per column after the barrier
  // would serialise one memory latency per column: the compiler cannot move such loads above the output stores.
  const int S = c.S;
  const int tok0 = c.tm * TOK, tok_hi = min(TOK, c.M - tok0);
  const int U = (tok_hi + 7) >> 3;  // units of 8 token columns that hold tokens
  const int own_max = (U + S - 1) / S;
  const int rank = static_cast<int>(c.rank);
  const int own_lo = rank * U / S, own_hi = (rank + 1) * U / S;
  const int row = q * 32 + lane;  // weight row of the tile = tensor-memory lane
  const int n = c.tn * 128 + row;
  const bool f32 = c.out_dtype == BITRL_OUT_F32;
  for (int j = ep; j < TOK; j += 128) {
    const int tok = tok0 + j;
    ptx::sts32(c.sc_addr + 4 * j, __float_as_uint(tok < c.M ? out_scale(c.mul, c.absmax[tok]) : 0.0f));
    ptx::sts32(c.rs_addr + 4 * j, static_cast<uint32_t>((tok < c.M && c.rowsum) ? c.rowsum[tok] : 0));
  }
  const bool use_res = c.residual && !f32;
  auto load_res = [&](int u, unsigned short (&r)[8]) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int col = u * 8 + j;
      r[j] = (use_res && col < tok_hi) ? c.residual[static_cast<size_t>(tok0 + col) * c.N + n] : static_cast<unsigned short>(0);
    }
  };
  unsigned short rcur[8] = {}, rnxt[8] = {};
  if (own_lo < own_hi) load_res(own_lo, rcur);
  // (the named barrier also publishes the scales among the four warps)
  const bool got = ptx::bar_red_and(1, 128, wait_acc());
  if (got) {
    // Send every peer the partial sums of its token columns: lane = weight row, so the 32 lanes of a warp store 128
    // consecutive bytes of the peer's receive area [sender slot][unit][column of the unit][row].
    ptx::tc_fence_after_sync();
    for (int i = 1; i < S; ++i) {
      const int p = (rank + i) % S;  // start with the next rank: spreads the traffic
      const int u_lo = p * U / S, u_hi = (p + 1) * U / S;
      const int slot = rank < p ? rank : rank - 1;
      const uint32_t dst = ptx::mapa_u32(c.recv_base + static_cast<uint32_t>(slot * own_max) * 4096u +
                                             static_cast<uint32_t>(row) * 4u, static_cast<uint32_t>(p));
      for (int u = u_lo; u < u_hi; ++u) {
        uint32_t v[8];
        ptx::tmem_ld_32x32b_x8(c.acc_tmem + static_cast<uint32_t>(u * 8) + (static_cast<uint32_t>(q * 32) << 16), v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 8; ++j) ptx::sts32_cluster(dst + static_cast<uint32_t>((u - u_lo) * 8 + j) * 512u, v[j]);
      }
    }
  }
  // Every partial sum has arrived once all threads of the cluster have passed this barrier (release / acquire at
  // cluster scope; the other warps of the CTA take part from the kernel's teardown).  Nobody writes to a peer after it.
  ptx::cluster_sync_all();
  if (got && !*c.failed) {
    // own partial sums + the S - 1 received ones, then the usual epilogue on this CTA's token columns
    for (int u = own_lo; u < own_hi; ++u) {
      if (u + 1 < own_hi) load_res(u + 1, rnxt);
      uint32_t v[8];
      ptx::tmem_ld_32x32b_x8(c.acc_tmem + static_cast<uint32_t>(u * 8) + (static_cast<uint32_t>(q * 32) << 16), v);
      ptx::tmem_ld_wait();
      for (int sl = 0; sl < S - 1; ++sl) {
        const uint32_t src = c.recv_base + static_cast<uint32_t>((sl * own_max + (u - own_lo)) * 8) * 512u +
                             static_cast<uint32_t>(row) * 4u;
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] += ptx::lds32(src + static_cast<uint32_t>(j) * 512u);
      }
      const uint4 rsa = ptx::lds128(c.rs_addr + u * 32), rsb = ptx::lds128(c.rs_addr + u * 32 + 16);
      const uint4 sca = ptx::lds128(c.sc_addr + u * 32), scb = ptx::lds128(c.sc_addr + u * 32 + 16);
      const uint32_t rsv[8] = {rsa.x, rsa.y, rsa.z, rsa.w, rsb.x, rsb.y, rsb.z, rsb.w};
      const uint32_t scv[8] = {sca.x, sca.y, sca.z, sca.w, scb.x, scb.y, scb.z, scb.w};
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int col = u * 8 + j;
        if (col < tok_hi) {
          const size_t off = static_cast<size_t>(tok0 + col) * c.N + n;
          const int acc = static_cast<int>(v[j] - rsv[j]);
          if (c.acc_out) c.acc_out[off] = acc;
          const float yv = __fmul_rn(static_cast<float>(acc), __uint_as_float(scv[j]));
          if (f32) {
            static_cast<float*>(c.y)[off] = yv;
          } else {
            unsigned short b = float_to_bf16_bits(yv);
            if (c.residual) b = float_to_bf16_bits(__fadd_rn(bf16_bits_to_float(rcur[j]), bf16_bits_to_float(b)));
            static_cast<unsigned short*>(c.y)[off] = b;
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) rcur[j] = rnxt[j];
    }
    ptx::tc_fence_before_sync();
  }
  return got;
}

}  // namespace bitrl
