// Shared device/host helpers of the bitrl CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/bitrl.h"

namespace bitrl {

// Kernel-side weight layout ("tile layout"), produced once by bitrl_linear_create:
//   [N/128 row tiles][K/128 k blocks][128 rows][32 bytes]
// so that one (row tile, k block) is a contiguous 4 KB piece.  Inside every 32-bit word (16 consecutive k)
// the 2-bit codes are transposed relative to the canonical format: bit 8b+2i holds k = 4i+b.  Then
// (word >> 2i) & 0x03030303 yields the four codes k = 4i..4i+3 in byte lanes 0..3, i.e. 16 consecutive
// bytes of an int8 row after four shift+mask pairs.
constexpr int TILE_ROWS = 128;
constexpr int TILE_K = 128;
constexpr int TILE_ROW_BYTES = TILE_K / 4;             // 32
constexpr int TILE_BYTES = TILE_ROWS * TILE_ROW_BYTES;  // 4096

// Device status word: [0] = status (BITRL_OK / BITRL_ERR_TIMEOUT), [1] = stage id of the wait that expired.
__device__ int g_status[4] = {0, 0, 0, 0};

__device__ __forceinline__ void report_timeout(int stage) {
  if (atomicCAS(&g_status[0], 0, BITRL_ERR_TIMEOUT) == 0) g_status[1] = stage;
}

// Lets the next kernel in the stream start its set-up, then waits until everything before this kernel has completed
// and its memory is visible.
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ float bf16_bits_to_float(unsigned short h) {
  return __uint_as_float(static_cast<unsigned>(h) << 16);
}

// fp32 -> bf16 bits, round-to-nearest-even (finite inputs; NaN kept quiet).
__device__ __forceinline__ unsigned short float_to_bf16_bits(float f) {
  __nv_bfloat16 b = __float2bfloat16_rn(f);
  return __bfloat16_as_ushort(b);
}

// Per-token quantization step: q = clip(rint(x * inv), -128, 127) with one fp32 multiply, ties-to-even.
__device__ __forceinline__ int quant_code(float x, float inv) {
  float q = rintf(__fmul_rn(x, inv));
  q = fminf(fmaxf(q, -128.0f), 127.0f);
  return static_cast<int>(q);
}

// Output scale of token m: gamma * (a_m / 127), two single fp32 operations in this order.
__device__ __forceinline__ float out_scale(float gamma, float absmax) {
  return __fmul_rn(gamma, __fdiv_rn(absmax, 127.0f));
}

// acc + sum of four (unsigned byte of a) * (signed byte of b).
__device__ __forceinline__ int dp4a_u8s8(uint32_t a, int b, int acc) {
  int d;
  asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(acc));
  return d;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int warp_sum_i(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---- host side ------------------------------------------------------------------------------------
struct Linear {
  uint8_t* tiles;  // device, tile layout, N*K/4 bytes
  float* gamma;    // device, [1]
  int32_t N, K;
};

void count_launch(int n = 1);
bitrl_status cuda_fail(cudaError_t e);  // records the code, returns BITRL_ERR_CUDA
#define BITRL_CUDA(call)                                   \
  do {                                                     \
    cudaError_t e__ = (call);                              \
    if (e__ != cudaSuccess) return ::bitrl::cuda_fail(e__); \
  } while (0)

// Launch with programmatic stream serialization: the kernel may be scheduled while its predecessor in the stream is
// still draining, so launch latency and the kernel's own set-up overlap the predecessor's tail.  Such kernels call
// pdl_enter() before they touch any global memory other than constant weights.
template <class... KArgs, class... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Launchers implemented in the kernel files (all asynchronous on `st`).
bitrl_status launch_pack(const float* W, int N, int K, uint8_t* packed, float* gamma, void* ws, cudaStream_t st);
bitrl_status launch_retile(const uint8_t* packed, int N, int K, uint8_t* tiles, cudaStream_t st);
bitrl_status launch_quant_act(const void* x, int M, int K, int8_t* xq, float* absmax, int32_t* rowsum,
                              cudaStream_t st);
bitrl_status launch_rmsnorm_quant(const void* h, int T, int K, int8_t* xq, float* absmax, int32_t* rowsum,
                                  void* u_out, cudaStream_t st);
bitrl_status launch_vrepeat_rmsnorm_quant(const void* qkv, int T, int n_heads, int n_kv, int hd, int8_t* xq,
                                          float* absmax, int32_t* rowsum, void* u_out, cudaStream_t st);
bitrl_status launch_relu2gate_rmsnorm_quant(const void* gu, int T, int F, int8_t* xq, float* absmax,
                                            int32_t* rowsum, void* u_out, cudaStream_t st);
// M <= 16.  Either x (bf16, quantized in the prologue) or (xq, absmax) must be given.
bitrl_status launch_gemv(const Linear* w, const void* x, const int8_t* xq, const float* absmax, int M, void* y,
                         int out_dtype, const void* residual, int8_t* xq_out, float* absmax_out,
                         int32_t* acc_out, cudaStream_t st);
// Any M >= 1, tcgen05 path, already quantized input.  splitk_ws: nullptr or M*N int32 of scratch (see gemm.cuh).
bitrl_status launch_gemm(const Linear* w, const int8_t* xq, const float* absmax, const int32_t* rowsum, int M,
                         void* y, int out_dtype, const void* residual, int32_t* acc_out, cudaStream_t st,
                         int32_t* splitk_ws = nullptr);

}  // namespace bitrl
