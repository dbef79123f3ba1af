// a0: absmean scale, ternarize + pack (Eq. 2 with tau = (gamma+1e-5)/2), and the re-tiling of the canonical
// packed bytes into the kernel-side tile layout.  Offline: runs once per matrix of the frozen backbone.
#pragma once

#include "common.cuh"

namespace bitrl {

constexpr int ABSSUM_THREADS = 256;
constexpr int ABSSUM_MAX_BLOCKS = 1024;

// Stage 1 of gamma: block b sums |W| over its contiguous chunk in fp64 (fixed order inside the block:
// per-thread strided serial sums, then a shared-memory tree), one partial per block.
__global__ void __launch_bounds__(ABSSUM_THREADS) abssum_partial_kernel(const float* __restrict__ W,
                                                                        long long count, long long chunk,
                                                                        double* __restrict__ partial) {
  __shared__ double red[ABSSUM_THREADS];
  const long long lo = static_cast<long long>(blockIdx.x) * chunk;
  long long hi = lo + chunk;
  if (hi > count) hi = count;
  double s = 0.0;
  // chunk is a multiple of 4 and W is 16-byte aligned, so float4 loads stay aligned.
  for (long long i = lo + 4LL * threadIdx.x; i + 3 < hi; i += 4LL * ABSSUM_THREADS) {
    const float4 v = *reinterpret_cast<const float4*>(W + i);
    s += static_cast<double>(fabsf(v.x));
    s += static_cast<double>(fabsf(v.y));
    s += static_cast<double>(fabsf(v.z));
    s += static_cast<double>(fabsf(v.w));
  }
  red[threadIdx.x] = s;
  __syncthreads();
  for (int o = ABSSUM_THREADS / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) partial[blockIdx.x] = red[0];
}

// Stage 2 (one CTA): thread t adds partials t, t + 256, ... in that order, a shared-memory tree adds the 256 sums (a
// fixed order, so gamma is reproducible), and S/count is rounded to fp32 once.  One thread adding up to 1024 partials in a
// row, as this kernel first did, was a chain of dependent loads and fp64 adds: 30 us, longer than either pass over W.
__global__ void __launch_bounds__(ABSSUM_THREADS) abssum_final_kernel(const double* __restrict__ partial, int nparts,
                                                                      long long count, float* __restrict__ gamma) {
  __shared__ double red[ABSSUM_THREADS];
  double s = 0.0;
  for (int i = threadIdx.x; i < nparts; i += ABSSUM_THREADS) s += partial[i];
  red[threadIdx.x] = s;
  __syncthreads();
  for (int o = ABSSUM_THREADS / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *gamma = static_cast<float>(red[0] / static_cast<double>(count));
}

// Each thread turns 16 consecutive weights of a row into one canonical 32-bit word (4 bytes, k ascending,
// code of k in bits 2(k%4) of byte k/4).
__global__ void __launch_bounds__(256) ternarize_pack_kernel(const float* __restrict__ W, long long nwords,
                                                             const float* __restrict__ gamma,
                                                             uint32_t* __restrict__ packed) {
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= nwords) return;
  const float s = __fadd_rn(*gamma, 1e-5f);
  const float4* src = reinterpret_cast<const float4*>(W + 16 * i);
  uint32_t word = 0;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 v = src[q];
    const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float r = rintf(__fdiv_rn(e[j], s));
      r = fminf(fmaxf(r, -1.0f), 1.0f);
      const uint32_t code = static_cast<uint32_t>(static_cast<int>(r) + 1);
      word |= code << (8 * q + 2 * j);
    }
  }
  packed[i] = word;
}

// Canonical [N][K/4] bytes -> tile layout.  One thread per 32-bit word; inside the word the 4x4 grid of
// 2-bit fields is transposed (canonical bit 8b+2i = k 4b+i  ->  tile bit 8b+2i = k 4i+b).
__global__ void __launch_bounds__(256) retile_kernel(const uint32_t* __restrict__ packed, int N, int K,
                                                     uint32_t* __restrict__ tiles) {
  const long long nwords = static_cast<long long>(N) * K / 16;
  const long long o = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (o >= nwords) return;
  // destination coordinates of word o
  const int j = static_cast<int>(o & 7);                 // word within the 32-byte row piece
  const int r = static_cast<int>((o >> 3) & (TILE_ROWS - 1));
  const long long blk = o >> 10;                         // (row tile, k block), 1024 words per tile block
  const int kblocks = K / TILE_K;
  const int kb = static_cast<int>(blk % kblocks);
  const int nt = static_cast<int>(blk / kblocks);
  const long long n = static_cast<long long>(nt) * TILE_ROWS + r;
  const uint32_t src = packed[n * (K / 16) + kb * 8 + j];
  uint32_t dst = 0;
#pragma unroll
  for (int b = 0; b < 4; ++b)
#pragma unroll
    for (int i = 0; i < 4; ++i) dst |= ((src >> (8 * b + 2 * i)) & 3u) << (8 * i + 2 * b);
  tiles[o] = dst;
}

inline int abssum_blocks(long long count) {
  long long b = (count + 16383) / 16384;
  if (b < 1) b = 1;
  if (b > ABSSUM_MAX_BLOCKS) b = ABSSUM_MAX_BLOCKS;
  return static_cast<int>(b);
}

bitrl_status launch_pack(const float* W, int N, int K, uint8_t* packed, float* gamma, void* ws, cudaStream_t st) {
  const long long count = static_cast<long long>(N) * K;
  const int nb = abssum_blocks(count);
  long long chunk = (count + nb - 1) / nb;
  chunk = (chunk + 3) & ~3LL;
  double* partial = static_cast<double*>(ws);
  abssum_partial_kernel<<<nb, ABSSUM_THREADS, 0, st>>>(W, count, chunk, partial);
  abssum_final_kernel<<<1, ABSSUM_THREADS, 0, st>>>(partial, nb, count, gamma);
  const long long nwords = count / 16;
  ternarize_pack_kernel<<<static_cast<unsigned>((nwords + 255) / 256), 256, 0, st>>>(
      W, nwords, gamma, reinterpret_cast<uint32_t*>(packed));
  count_launch(3);
  BITRL_CUDA(cudaGetLastError());
  return BITRL_OK;
}

bitrl_status launch_retile(const uint8_t* packed, int N, int K, uint8_t* tiles, cudaStream_t st) {
  const long long nwords = static_cast<long long>(N) * K / 16;
  retile_kernel<<<static_cast<unsigned>((nwords + 255) / 256), 256, 0, st>>>(
      reinterpret_cast<const uint32_t*>(packed), N, K, reinterpret_cast<uint32_t*>(tiles));
  count_launch(1);
  BITRL_CUDA(cudaGetLastError());
  return BITRL_OK;
}

}  // namespace bitrl
