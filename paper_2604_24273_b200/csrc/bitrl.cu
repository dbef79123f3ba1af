// C-ABI entry points of the bitrl library (declared and documented in include/bitrl.h).  Host code here only
// validates arguments, carves workspaces and launches the kernels of pack.cuh / quant.cuh / gemv.cuh / gemm.cuh.
#include <atomic>
#include <cstdlib>
#include <new>
#include <vector>

#include "common.cuh"

namespace bitrl {
static std::atomic<uint64_t> g_launches{0};
static std::atomic<int> g_last_cuda{0};
static std::atomic<int> g_last_stage{0};

void count_launch(int n) { g_launches.fetch_add(static_cast<uint64_t>(n), std::memory_order_relaxed); }
bitrl_status cuda_fail(cudaError_t e) {
  g_last_cuda.store(static_cast<int>(e));
  (void)cudaGetLastError();
  return BITRL_ERR_CUDA;
}

// Which operand path the GEMM uses for the expanded weights; BITRL_GEMM_A=smem selects the shared-memory one.
bool gemm_a_in_tmem() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("BITRL_GEMM_A");
    v = (e && e[0] == 's') ? 0 : 1;
  }
  return v == 1;
}

// BITRL_GEMM_PAIR=1 forces the paired-CTA GEMM wherever the shape allows it, 0 forbids it (tuning and fallback knob).
int gemm_pair_mode() {
  static int v = -2;
  if (v == -2) {
    const char* e = getenv("BITRL_GEMM_PAIR");
    v = !e ? -1 : (e[0] == '1' ? 1 : 0);
  }
  return v;
}

// BITRL_GEMM_CLSK=0 turns the cluster split-K GEMM off (split launches then go through scratch and a finishing kernel);
// a value of 2 ... 8 makes every launch that can take a cluster of that size take it (tuning runs).
int gemm_clsk_mode() {
  static int v = -2;
  if (v == -2) {
    const char* e = getenv("BITRL_GEMM_CLSK");
    v = !e ? -1 : atoi(e);
  }
  return v;
}

// BITRL_GEMM_TOK=<64|128|192|224|256> overrides the launcher's choice of token-tile width (for tuning runs).
int gemm_forced_tok() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("BITRL_GEMM_TOK");
    const int t = e ? atoi(e) : 0;
    v = (t == 64 || t == 128 || t == 192 || t == 224 || t == 256) ? t : 0;
  }
  return v;
}

// Largest M that a call with pre-quantized activations gives to the streaming kernel; above it the tensor-core GEMM
// (with its cluster split-K) is faster.  BITRL_GEMV_Q_MAX_M=<1..16> overrides it (tuning runs).
constexpr int GEMV_Q_MAX_M_DEFAULT = 4;
int gemv_q_max_m() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("BITRL_GEMV_Q_MAX_M");
    const int t = e ? atoi(e) : 0;
    v = (t >= 1 && t <= BITRL_GEMV_MAX_M) ? t : GEMV_Q_MAX_M_DEFAULT;
  }
  return v;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

// The kernels are compiled for sm_100a only; any other device cannot run them.
static bitrl_status check_arch() {
  static int ok[64] = {0};
  int dev = 0;
  BITRL_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return BITRL_ERR_ARCH;
  if (ok[dev] == 0) {
    int major = 0, minor = 0;
    BITRL_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    BITRL_CUDA(cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev));
    ok[dev] = (major == 10 && minor == 0) ? 1 : -1;
  }
  return ok[dev] == 1 ? BITRL_OK : BITRL_ERR_ARCH;
}
}  // namespace bitrl

#include "pack.cuh"
#include "quant.cuh"
#include "gemv.cuh"
#include "gemv_multi.cuh"
#include "gemm.cuh"
#include "attention.cuh"
#include "heads.cuh"
#include "gemm_w8.cuh"
#include "w4.cuh"
#include "gemv5.cuh"
#include "gemv8_multi.cuh"

using namespace bitrl;

struct bitrl_linear {
  Linear l;
};

struct bitrl_linear5 {
  Linear5 l;
};

struct bitrl_encoder {
  std::vector<const bitrl_linear*> layers;  // 4 per block: qkv, out, gateup, down
  int L, d, d_ff, n_heads, n_kv_heads, head_dim;
};

namespace {

inline bool shape_ok(int N, int K) { return N >= 128 && K >= 128 && N % 128 == 0 && K % 128 == 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Workspace of the M > 16 path: x_q [M,K] int8, absmax [M] f32, rowsum [M] i32, and for small M the split-K scratch
// [M,N] int32.
struct FwdWs {
  int8_t* xq;
  float* absmax;
  int32_t* rowsum;
  int32_t* splitk;
  size_t bytes;
};
inline FwdWs carve_fwd(void* ws, int M, int K, int N) {
  FwdWs f;
  size_t off = 0;
  unsigned char* b = static_cast<unsigned char*>(ws);
  f.xq = reinterpret_cast<int8_t*>(b + off);
  off += align_up(static_cast<size_t>(M) * K, 256);
  f.absmax = reinterpret_cast<float*>(b + off);
  off += align_up(static_cast<size_t>(M) * 4, 256);
  f.rowsum = reinterpret_cast<int32_t*>(b + off);
  off += align_up(static_cast<size_t>(M) * 4, 256);
  f.splitk = nullptr;
  if (M <= GM_SPLITK_MAX_M) {
    f.splitk = reinterpret_cast<int32_t*>(b + off);
    off += align_up(static_cast<size_t>(M) * N * 4, 256);
  }
  f.bytes = off;
  return f;
}

}  // namespace

extern "C" {

size_t bitrl_pack_workspace_bytes(int32_t N, int32_t K) {
  (void)N; (void)K;
  return ABSSUM_MAX_BLOCKS * sizeof(double);
}

bitrl_status bitrl_pack_ternary(const float* W, int32_t N, int32_t K, uint8_t* packed, float* gamma,
                                void* workspace, size_t workspace_bytes, void* stream) {
  if (!W || !packed || !gamma) return BITRL_ERR_NULL;
  if (!shape_ok(N, K)) return BITRL_ERR_SHAPE;
  if (!aligned16(W) || !aligned16(packed) || !aligned16(workspace)) return BITRL_ERR_ALIGN;
  if (!workspace || workspace_bytes < bitrl_pack_workspace_bytes(N, K)) return BITRL_ERR_WORKSPACE;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_pack(W, N, K, packed, gamma, workspace, static_cast<cudaStream_t>(stream));
}

}  // extern "C"

// Scratch of bitrl_pack_ternary_static: one fp64 partial sum per reduction block.  It is part of the library
// image, so every GPU that loads the library holds these 8 KB until the process exits.  In host code the name
// below is only a handle for cudaGetSymbolAddress, never a pointer a kernel could use.
static __device__ __align__(256) double g_pack_static_scratch[ABSSUM_MAX_BLOCKS];

extern "C" {

bitrl_status bitrl_pack_ternary_static(const float* W, int32_t N, int32_t K, uint8_t* packed, float* gamma,
                                       void* stream) {
  if (!W || !packed || !gamma) return BITRL_ERR_NULL;
  if (!shape_ok(N, K)) return BITRL_ERR_SHAPE;
  if (static_cast<long long>(N) * K > BITRL_PACK_STATIC_MAX_WEIGHTS) return BITRL_ERR_LIMIT;
  if (!aligned16(W) || !aligned16(packed)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  // Device address of the scratch array, looked up once per device with that device current.
  static double* scratch_addr[64] = {nullptr};
  int dev = 0;
  BITRL_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return BITRL_ERR_ARCH;
  if (!scratch_addr[dev]) {
    double* p = nullptr;
    BITRL_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_pack_static_scratch));
    if (!p) return BITRL_ERR_CUDA;
    scratch_addr[dev] = p;
  }
  // The reduction writes partial[0 .. blocks) before its last stage reads exactly those slots, so stale
  // contents from an earlier call are never observed and nothing needs clearing.
  return launch_pack(W, N, K, packed, gamma, scratch_addr[dev], static_cast<cudaStream_t>(stream));
}

bitrl_status bitrl_linear_create(const uint8_t* packed, const float* gamma, int32_t N, int32_t K,
                                 bitrl_linear_t** out, void* stream) {
  if (!packed || !gamma || !out) return BITRL_ERR_NULL;
  if (!shape_ok(N, K)) return BITRL_ERR_SHAPE;
  if (!aligned16(packed)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  bitrl_linear* w = new (std::nothrow) bitrl_linear();
  if (!w) return BITRL_ERR_CUDA;
  w->l.N = N;
  w->l.K = K;
  w->l.tiles = nullptr;
  w->l.gamma = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMalloc(&w->l.tiles, static_cast<size_t>(N) * K / 4);
  if (e == cudaSuccess) e = cudaMalloc(&w->l.gamma, 256);
  if (e == cudaSuccess) e = cudaMemcpyAsync(w->l.gamma, gamma, sizeof(float), cudaMemcpyDeviceToDevice, st);
  if (e != cudaSuccess) {
    cudaFree(w->l.tiles);
    cudaFree(w->l.gamma);
    delete w;
    return cuda_fail(e);
  }
  s = launch_retile(packed, N, K, w->l.tiles, st);
  // The handle is complete when this returns: the forward kernels prefetch weights ahead of their stream dependencies.
  if (s == BITRL_OK && cudaStreamSynchronize(st) != cudaSuccess) s = cuda_fail(cudaGetLastError());
  if (s != BITRL_OK) {
    cudaFree(w->l.tiles);
    cudaFree(w->l.gamma);
    delete w;
    return s;
  }
  *out = w;
  return BITRL_OK;
}

bitrl_status bitrl_linear_destroy(bitrl_linear_t* w) {
  if (!w) return BITRL_OK;
  cudaFree(w->l.tiles);
  cudaFree(w->l.gamma);
  delete w;
  return BITRL_OK;
}

bitrl_status bitrl_quant_act(const void* x, int32_t M, int32_t K, int8_t* xq, float* absmax, int32_t* rowsum,
                             void* stream) {
  if (!x || !xq || !absmax) return BITRL_ERR_NULL;
  if (M < 1 || K < 128 || K % 128 != 0) return BITRL_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(xq)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_quant_act(x, M, K, xq, absmax, rowsum, static_cast<cudaStream_t>(stream));
}

// Whole-layer calls: up to this M the streaming kernel (quantization in its prologue) is the faster form; from there to
// BITRL_GEMV_MAX_M it still serves callers that pass no workspace, but quantizer + tensor-core GEMM is faster (a block's
// four layers at M = 8: 31 against 44 us; at M = 16: 2-3 x).
constexpr int FWD_GEMV_PREFERRED_MAX_M = 4;

size_t bitrl_workspace_bytes(int32_t M, int32_t K, int32_t N) {
  if (M < 1 || K < 1 || N < 1) return 0;
  if (M <= FWD_GEMV_PREFERRED_MAX_M && gemv_fits(M, K)) return 0;
  return carve_fwd(nullptr, M, K, N).bytes;
}

static bitrl_status forward_impl(const bitrl_linear_t* w, const void* x, int32_t M, int32_t K, int32_t N, void* y,
                                 int32_t out_dtype, void* workspace, size_t workspace_bytes, int8_t* xq_out,
                                 float* absmax_out, int32_t* acc_out, bool debug, void* stream) {
  if (!w || !x || !y) return BITRL_ERR_NULL;
  if (M < 1 || K != w->l.K || N != w->l.N) return BITRL_ERR_SHAPE;
  if (out_dtype != BITRL_OUT_F32 && out_dtype != BITRL_OUT_BF16) return BITRL_ERR_DTYPE;
  if (!aligned16(x) || !aligned16(y)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t need = carve_fwd(nullptr, M, K, N).bytes;
  if (gemv_fits(M, K) && (M <= FWD_GEMV_PREFERRED_MAX_M || !workspace || workspace_bytes < need))
    return launch_gemv(&w->l, x, nullptr, nullptr, M, y, out_dtype, nullptr, xq_out, absmax_out, acc_out, st);
  if (!workspace || workspace_bytes < need) return BITRL_ERR_WORKSPACE;
  if (!aligned16(workspace)) return BITRL_ERR_ALIGN;
  FwdWs f = carve_fwd(workspace, M, K, N);
  s = launch_quant_act(x, M, K, f.xq, f.absmax, f.rowsum, st);
  if (s != BITRL_OK) return s;
  s = launch_gemm(&w->l, f.xq, f.absmax, f.rowsum, M, y, out_dtype, nullptr, acc_out, st, f.splitk);
  if (s != BITRL_OK) return s;
  if (debug) {
    if (xq_out) BITRL_CUDA(cudaMemcpyAsync(xq_out, f.xq, static_cast<size_t>(M) * K, cudaMemcpyDeviceToDevice, st));
    if (absmax_out)
      BITRL_CUDA(cudaMemcpyAsync(absmax_out, f.absmax, static_cast<size_t>(M) * 4, cudaMemcpyDeviceToDevice, st));
  }
  return BITRL_OK;
}

bitrl_status bitrl_bitlinear_forward(const bitrl_linear_t* w, const void* x, int32_t M, int32_t K, int32_t N,
                                     void* y, int32_t out_dtype, void* workspace, size_t workspace_bytes,
                                     void* stream) {
  return forward_impl(w, x, M, K, N, y, out_dtype, workspace, workspace_bytes, nullptr, nullptr, nullptr, false,
                      stream);
}

bitrl_status bitrl_bitlinear_forward_multi(int32_t count, const bitrl_linear_t* const* w, const void* const* x,
                                           void* const* y, int32_t M, int32_t out_dtype, void* stream) {
  if (!w || !x || !y) return BITRL_ERR_NULL;
  if (count < 1 || count > BITRL_MULTI_MAX_JOBS || M < 1 || M > BITRL_GEMV_MAX_M) return BITRL_ERR_SHAPE;
  if (out_dtype != BITRL_OUT_F32 && out_dtype != BITRL_OUT_BF16) return BITRL_ERR_DTYPE;
  const Linear* lins[BITRL_MULTI_MAX_JOBS];
  for (int i = 0; i < count; ++i) {
    if (!w[i] || !x[i] || !y[i]) return BITRL_ERR_NULL;
    if (!aligned16(x[i]) || !aligned16(y[i])) return BITRL_ERR_ALIGN;
    lins[i] = &w[i]->l;
  }
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_gemv_multi(count, lins, x, y, M, out_dtype, static_cast<cudaStream_t>(stream));
}

bitrl_status bitrl_bitlinear_forward_debug(const bitrl_linear_t* w, const void* x, int32_t M, int32_t K,
                                           int32_t N, void* y, int32_t out_dtype, void* workspace,
                                           size_t workspace_bytes, int8_t* xq_out, float* absmax_out,
                                           int32_t* acc_out, void* stream) {
  return forward_impl(w, x, M, K, N, y, out_dtype, workspace, workspace_bytes, xq_out, absmax_out, acc_out, true,
                      stream);
}

bitrl_status bitrl_bitlinear_forward_q(const bitrl_linear_t* w, const int8_t* xq, const float* absmax,
                                       const int32_t* rowsum, int32_t M, void* y, int32_t out_dtype,
                                       const void* residual, int32_t* acc_out, void* stream) {
  if (!w || !xq || !absmax || !rowsum || !y) return BITRL_ERR_NULL;
  if (M < 1) return BITRL_ERR_SHAPE;
  if (out_dtype != BITRL_OUT_F32 && out_dtype != BITRL_OUT_BF16) return BITRL_ERR_DTYPE;
  if (residual && out_dtype != BITRL_OUT_BF16) return BITRL_ERR_DTYPE;
  if (!aligned16(xq) || !aligned16(y) || !aligned16(residual)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (M <= gemv_q_max_m() && gemv_fits(M, w->l.K))
    return launch_gemv(&w->l, nullptr, xq, absmax, M, y, out_dtype, residual, nullptr, nullptr, acc_out, st);
  return launch_gemm(&w->l, xq, absmax, rowsum, M, y, out_dtype, residual, acc_out, st);
}

bitrl_status bitrl_rmsnorm_quant(const void* h, int32_t T, int32_t K, int8_t* xq, float* absmax,
                                 int32_t* rowsum, void* u_out, void* stream) {
  if (!h || !xq || !absmax) return BITRL_ERR_NULL;
  if (T < 1 || K < 128 || K % 128 != 0 || K > 49152) return BITRL_ERR_SHAPE;
  if (!aligned16(h) || !aligned16(xq) || !aligned16(u_out)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_rmsnorm_quant(h, T, K, xq, absmax, rowsum, u_out, static_cast<cudaStream_t>(stream));
}

bitrl_status bitrl_vrepeat_rmsnorm_quant(const void* qkv, int32_t T, int32_t n_heads, int32_t n_kv_heads,
                                         int32_t head_dim, int8_t* xq, float* absmax, int32_t* rowsum,
                                         void* u_out, void* stream) {
  if (!qkv || !xq || !absmax) return BITRL_ERR_NULL;
  if (T < 1 || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads != 0 || head_dim < 8 || head_dim % 8 != 0 ||
      (n_kv_heads * head_dim) % 128 != 0 || (n_heads * head_dim) % 128 != 0)
    return BITRL_ERR_SHAPE;
  if (!aligned16(qkv) || !aligned16(xq) || !aligned16(u_out)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_vrepeat_rmsnorm_quant(qkv, T, n_heads, n_kv_heads, head_dim, xq, absmax, rowsum, u_out,
                                      static_cast<cudaStream_t>(stream));
}

bitrl_status bitrl_relu2gate_rmsnorm_quant(const void* gu, int32_t T, int32_t F, int8_t* xq, float* absmax,
                                           int32_t* rowsum, void* u_out, void* stream) {
  if (!gu || !xq || !absmax) return BITRL_ERR_NULL;
  if (T < 1 || F < 128 || F % 128 != 0 || F > 49152) return BITRL_ERR_SHAPE;
  if (!aligned16(gu) || !aligned16(xq) || !aligned16(u_out)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_relu2gate_rmsnorm_quant(gu, T, F, xq, absmax, rowsum, u_out, static_cast<cudaStream_t>(stream));
}

// ---- encoder ------------------------------------------------------------------------------------------

bitrl_status bitrl_encoder_create(const bitrl_linear_t* const* layers, int32_t L, int32_t d, int32_t d_ff,
                                  int32_t n_heads, int32_t n_kv_heads, bitrl_encoder_t** enc) {
  if (!layers || !enc) return BITRL_ERR_NULL;
  if (L < 1 || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads != 0 || d % n_heads != 0) return BITRL_ERR_SHAPE;
  const int hd = d / n_heads;
  const int n_qkv = d + 2 * n_kv_heads * hd;
  if (!shape_ok(d, d_ff) || n_qkv % 128 != 0 || (n_kv_heads * hd) % 128 != 0 || hd % 8 != 0) return BITRL_ERR_SHAPE;
  for (int l = 0; l < L; ++l) {
    const bitrl_linear_t* const* q = layers + 4 * l;
    for (int j = 0; j < 4; ++j)
      if (!q[j]) return BITRL_ERR_NULL;
    if (q[0]->l.K != d || q[0]->l.N != n_qkv) return BITRL_ERR_SHAPE;
    if (q[1]->l.K != d || q[1]->l.N != d) return BITRL_ERR_SHAPE;
    if (q[2]->l.K != d || q[2]->l.N != 2 * d_ff) return BITRL_ERR_SHAPE;
    if (q[3]->l.K != d_ff || q[3]->l.N != d) return BITRL_ERR_SHAPE;
  }
  bitrl_encoder* e = new (std::nothrow) bitrl_encoder();
  if (!e) return BITRL_ERR_CUDA;
  e->layers.assign(layers, layers + 4 * L);
  e->L = L; e->d = d; e->d_ff = d_ff; e->n_heads = n_heads; e->n_kv_heads = n_kv_heads; e->head_dim = hd;
  *enc = e;
  return BITRL_OK;
}

bitrl_status bitrl_encoder_destroy(bitrl_encoder_t* enc) {
  delete enc;
  return BITRL_OK;
}

namespace {
struct EncWs {
  int8_t* xq;       // [T, max(d, d_ff)]
  float* absmax;    // [T]
  int32_t* rowsum;  // [T]
  unsigned short* wide;  // [T, max(n_qkv, 2 d_ff)] bf16: qkv, then gate/up
  int32_t* splitk;       // [T, max N] int32 split-K scratch of the GEMM (only for small T)
  unsigned short* att;   // [T, d] bf16 attention output (only with real attention)
  float2* rope;          // [max_state_len, head_dim/2] rotary table (only with real attention)
  size_t bytes;
};
EncWs carve_enc(void* ws, const bitrl_encoder* e, int T, int max_state_len) {
  EncWs w;
  size_t off = 0;
  unsigned char* b = static_cast<unsigned char*>(ws);
  const int kmax = e->d > e->d_ff ? e->d : e->d_ff;
  const int n_qkv = e->d + 2 * e->n_kv_heads * e->head_dim;
  const int wmax = n_qkv > 2 * e->d_ff ? n_qkv : 2 * e->d_ff;
  w.xq = reinterpret_cast<int8_t*>(b + off);
  off += align_up(static_cast<size_t>(T) * kmax, 256);
  w.absmax = reinterpret_cast<float*>(b + off);
  off += align_up(static_cast<size_t>(T) * 4, 256);
  w.rowsum = reinterpret_cast<int32_t*>(b + off);
  off += align_up(static_cast<size_t>(T) * 4, 256);
  w.wide = reinterpret_cast<unsigned short*>(b + off);
  off += align_up(static_cast<size_t>(T) * wmax * 2, 256);
  w.splitk = nullptr;
  if (T <= GM_SPLITK_MAX_M) {
    w.splitk = reinterpret_cast<int32_t*>(b + off);
    off += align_up(static_cast<size_t>(T) * wmax * 4, 256);
  }
  w.att = nullptr;
  w.rope = nullptr;
  if (max_state_len > 0) {
    w.att = reinterpret_cast<unsigned short*>(b + off);
    off += align_up(static_cast<size_t>(T) * e->d * 2, 256);
    w.rope = reinterpret_cast<float2*>(b + off);
    off += rope_table_bytes(max_state_len, e->head_dim);
  }
  w.bytes = off;
  return w;
}

bool attention_shape_ok(int n_heads, int n_kv_heads, int head_dim, int max_state_len) {
  return n_heads >= 1 && n_kv_heads >= 1 && n_heads % n_kv_heads == 0 && (head_dim == 64 || head_dim == 128) &&
         max_state_len >= 1 && max_state_len <= BITRL_ATTN_MAX_STATE_TOKENS;
}

// One pass over the blocks.  max_state_len == 0: identity attention (V repeated); else real attention per state.
bitrl_status encoder_run(const bitrl_encoder_t* enc, const void* h_in, int32_t T, const int32_t* state_off,
                         int32_t n_states, int32_t max_state_len, double theta, void* h_out, void* pooled,
                         void* workspace, cudaStream_t st) {
  bitrl_status s;
  EncWs w = carve_enc(workspace, enc, T, max_state_len);
  const int d = enc->d, F = enc->d_ff;
  if (h_out != h_in)
    BITRL_CUDA(cudaMemcpyAsync(h_out, h_in, static_cast<size_t>(T) * d * 2, cudaMemcpyDeviceToDevice, st));
  if (max_state_len > 0 && (s = launch_rope_table(w.rope, max_state_len, enc->head_dim, theta, st)) != BITRL_OK) return s;
  auto linear = [&](const bitrl_linear* lin, void* y, const void* residual) -> bitrl_status {
    if (T <= gemv_q_max_m() && gemv_fits(T, lin->l.K))
      return launch_gemv(&lin->l, nullptr, w.xq, w.absmax, T, y, BITRL_OUT_BF16, residual, nullptr, nullptr, nullptr, st);
    return launch_gemm(&lin->l, w.xq, w.absmax, w.rowsum, T, y, BITRL_OUT_BF16, residual, nullptr, st, w.splitk);
  };
  for (int l = 0; l < enc->L; ++l) {
    const bitrl_linear* const* q = enc->layers.data() + 4 * l;
    if ((s = launch_rmsnorm_quant(h_out, T, d, w.xq, w.absmax, w.rowsum, nullptr, st)) != BITRL_OK) return s;
    if ((s = linear(q[0], w.wide, nullptr)) != BITRL_OK) return s;
    if (max_state_len > 0) {
      if ((s = launch_attention(w.wide, T, state_off, n_states, max_state_len, enc->n_heads, enc->n_kv_heads,
                                enc->head_dim, w.rope, w.att, st)) != BITRL_OK) return s;
      if ((s = launch_rmsnorm_quant(w.att, T, d, w.xq, w.absmax, w.rowsum, nullptr, st)) != BITRL_OK) return s;
    } else {
      if ((s = launch_vrepeat_rmsnorm_quant(w.wide, T, enc->n_heads, enc->n_kv_heads, enc->head_dim, w.xq, w.absmax,
                                            w.rowsum, nullptr, st)) != BITRL_OK) return s;
    }
    if ((s = linear(q[1], h_out, h_out)) != BITRL_OK) return s;
    if ((s = launch_rmsnorm_quant(h_out, T, d, w.xq, w.absmax, w.rowsum, nullptr, st)) != BITRL_OK) return s;
    if ((s = linear(q[2], w.wide, nullptr)) != BITRL_OK) return s;
    if ((s = launch_relu2gate_rmsnorm_quant(w.wide, T, F, w.xq, w.absmax, w.rowsum, nullptr, st)) != BITRL_OK) return s;
    if ((s = linear(q[3], h_out, h_out)) != BITRL_OK) return s;
  }
  if (pooled) return launch_pool_last_token(h_out, T, state_off, n_states, max_state_len, d, pooled, st);
  return BITRL_OK;
}
}  // namespace

size_t bitrl_encoder_workspace_bytes(const bitrl_encoder_t* enc, int32_t T) {
  if (!enc || T < 1) return 0;
  return carve_enc(nullptr, enc, T, 0).bytes;
}

bitrl_status bitrl_encoder_forward(const bitrl_encoder_t* enc, const void* h_in, int32_t T, void* h_out,
                                   void* workspace, size_t workspace_bytes, void* stream) {
  if (!enc || !h_in || !h_out) return BITRL_ERR_NULL;
  if (T < 1) return BITRL_ERR_SHAPE;
  if (!workspace || workspace_bytes < bitrl_encoder_workspace_bytes(enc, T)) return BITRL_ERR_WORKSPACE;
  if (!aligned16(h_in) || !aligned16(h_out) || !aligned16(workspace)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return encoder_run(enc, h_in, T, nullptr, 0, 0, 0.0, h_out, nullptr, workspace, static_cast<cudaStream_t>(stream));
}

size_t bitrl_encoder_states_workspace_bytes(const bitrl_encoder_t* enc, int32_t T, int32_t max_state_len) {
  if (!enc || T < 1 || max_state_len < 1) return 0;
  return carve_enc(nullptr, enc, T, max_state_len).bytes;
}

bitrl_status bitrl_encoder_forward_states(const bitrl_encoder_t* enc, const void* h_in, int32_t T,
                                          const int32_t* state_off, int32_t n_states, int32_t max_state_len,
                                          double theta, void* h_out, void* pooled, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  if (!enc || !h_in || !h_out) return BITRL_ERR_NULL;
  if (T < 1 || n_states < 1 || !(theta > 0.0)) return BITRL_ERR_SHAPE;
  if (!attention_shape_ok(enc->n_heads, enc->n_kv_heads, enc->head_dim, max_state_len)) return BITRL_ERR_SHAPE;
  if (!state_off && static_cast<long long>(n_states) * max_state_len != T) return BITRL_ERR_SHAPE;
  if (!workspace || workspace_bytes < bitrl_encoder_states_workspace_bytes(enc, T, max_state_len))
    return BITRL_ERR_WORKSPACE;
  if (!aligned16(h_in) || !aligned16(h_out) || !aligned16(workspace) || !aligned16(pooled)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return encoder_run(enc, h_in, T, state_off, n_states, max_state_len, theta, h_out, pooled, workspace,
                     static_cast<cudaStream_t>(stream));
}

// ---- attention inside each state, last-token pooling ------------------------------------------------------

size_t bitrl_attention_workspace_bytes(int32_t max_state_len, int32_t head_dim) {
  if (max_state_len < 1 || head_dim < 2) return 0;
  return rope_table_bytes(max_state_len, head_dim);
}

bitrl_status bitrl_attention(const void* qkv, int32_t T, const int32_t* state_off, int32_t n_states,
                             int32_t max_state_len, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                             double theta, void* att, void* workspace, size_t workspace_bytes, void* stream) {
  if (!qkv || !att) return BITRL_ERR_NULL;
  if (T < 1 || n_states < 1 || !(theta > 0.0)) return BITRL_ERR_SHAPE;
  if (!attention_shape_ok(n_heads, n_kv_heads, head_dim, max_state_len)) return BITRL_ERR_SHAPE;
  if (!state_off && static_cast<long long>(n_states) * max_state_len != T) return BITRL_ERR_SHAPE;
  if (!workspace || workspace_bytes < bitrl_attention_workspace_bytes(max_state_len, head_dim)) return BITRL_ERR_WORKSPACE;
  if (!aligned16(qkv) || !aligned16(att) || !aligned16(workspace)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float2* rope = static_cast<float2*>(workspace);
  if ((s = launch_rope_table(rope, max_state_len, head_dim, theta, st)) != BITRL_OK) return s;
  return launch_attention(qkv, T, state_off, n_states, max_state_len, n_heads, n_kv_heads, head_dim, rope, att, st);
}

bitrl_status bitrl_pool_last_token(const void* h, int32_t T, const int32_t* state_off, int32_t n_states,
                                   int32_t max_state_len, int32_t d, void* out, void* stream) {
  if (!h || !out) return BITRL_ERR_NULL;
  if (T < 1 || n_states < 1 || max_state_len < 1 || d < 8 || d % 8 != 0) return BITRL_ERR_SHAPE;
  if (!state_off && static_cast<long long>(n_states) * max_state_len != T) return BITRL_ERR_SHAPE;
  if (!aligned16(h) || !aligned16(out)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_pool_last_token(h, T, state_off, n_states, max_state_len, d, out, static_cast<cudaStream_t>(stream));
}

// ---- heads, GAE, PPO objective ----------------------------------------------------------------------------

bitrl_status bitrl_heads_forward(const void* h, int32_t B, int32_t d, int32_t H1, int32_t H2, const bitrl_head_t* heads,
                                 int32_t n_heads, float* const* out, void* stream) {
  if (!h || !heads || !out) return BITRL_ERR_NULL;
  if (B < 1 || d < 16 || d % 16 != 0 || H1 < 1 || H1 > HEAD_MAX_WIDTH || H2 < 1 || H2 > HEAD_MAX_WIDTH || n_heads < 1 ||
      n_heads > HEAD_MAX_HEADS)
    return BITRL_ERR_SHAPE;
  HeadsArgs a;
  for (int i = 0; i < n_heads; ++i) {
    const bitrl_head_t& p = heads[i];
    if (!p.W1t || !p.b1 || !p.W2t || !p.b2 || !p.W3t || !p.b3 || !out[i]) return BITRL_ERR_NULL;
    if (p.n_out < 1 || p.n_out > HEAD_MAX_WIDTH) return BITRL_ERR_SHAPE;
    a.head[i] = p;
    a.out[i] = out[i];
  }
  for (int i = n_heads; i < HEAD_MAX_HEADS; ++i) { a.head[i] = heads[0]; a.out[i] = nullptr; }
  if (!aligned16(h)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  a.h = static_cast<const unsigned short*>(h);
  a.B = B; a.d = d; a.H1 = H1; a.H2 = H2;
  return launch_heads(a, n_heads, static_cast<cudaStream_t>(stream));
}

bitrl_status bitrl_gae(const float* rewards, const float* values, const float* dones, int32_t T, int32_t E, float gamma,
                       float lambda, float* adv, float* returns, void* stream) {
  if (!rewards || !values || !dones || !adv) return BITRL_ERR_NULL;
  if (T < 1 || E < 1) return BITRL_ERR_SHAPE;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  BITRL_CUDA(launch_pdl(gae_kernel, dim3((E + GAE_ENVS - 1) / GAE_ENVS), dim3(GAE_CHUNKS * GAE_ENVS), 0,
                        static_cast<cudaStream_t>(stream), rewards, values,
                        dones, T, E, gamma, lambda, adv, returns));
  count_launch(1);
  return BITRL_OK;
}

bitrl_status bitrl_ppo_loss(const float* logits, const int32_t* actions, const float* old_logp, const float* adv,
                            const float* values, const float* returns, int32_t B, int32_t A, float eps, float beta,
                            float* terms, float* dlogits, float* dvalues, float* summary, void* stream) {
  if (!logits || !actions || !old_logp || !adv || !values || !returns || !terms || !summary) return BITRL_ERR_NULL;
  if (B < 1 || A < 1) return BITRL_ERR_SHAPE;
  if (!aligned16(terms)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  PpoArgs a{logits, actions, old_logp, adv, values, returns, B, A, eps, beta, terms, dlogits, dvalues};
  BITRL_CUDA(launch_pdl(ppo_terms_kernel, dim3((B + 7) / 8), dim3(256), 0, st, a));
  BITRL_CUDA(launch_pdl(ppo_summary_kernel, dim3(1), dim3(256), 0, st, static_cast<const float*>(terms), B, beta, summary));
  count_launch(2);
  return BITRL_OK;
}

// ---- W8A8 layer of the higher-precision critic ----------------------------------------------------------------

bitrl_status bitrl_w8_quantize(const float* W, int32_t N, int32_t K, int8_t* wq, float* scale, void* stream) {
  if (!W || !wq || !scale) return BITRL_ERR_NULL;
  if (!shape_ok(N, K)) return BITRL_ERR_SHAPE;
  if (!aligned16(W) || !aligned16(wq)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_w8_quantize(W, N, K, wq, scale, static_cast<cudaStream_t>(stream));
}

// Critic layers: up to this M the streaming kernels are the faster form; from there to BITRL_GEMV_MAX_M they still serve
// callers that pass no workspace, but quantizer (+ expansion) + tensor-core GEMM is 1.2-3 x faster (measured at M = 8, 12, 16).
constexpr int W8_GEMV_PREFERRED_MAX_M = 4;
// ... and only for rows of up to this many weights: a warp of the streaming kernels walks whole rows, so long rows of a
// matrix with few rows leave it little memory parallelism (6912 -> 2560 at M = 1: 11.6 us streaming, 8.9 us through the
// GEMM and its cluster split-K; 2560 -> 6912: 6.1 against 9.0 us).
constexpr int W8_GEMV_PREFERRED_MAX_K = 4096;
static bool w8_streaming_preferred(int M, int K) {
  return M <= W8_GEMV_PREFERRED_MAX_M && K <= W8_GEMV_PREFERRED_MAX_K && gemv_w8_fits(M, K);
}
// The INT4 layer's GEMM form has a third launch (the expansion to int8), so its streaming kernel keeps long rows too
// (6912 -> 2560 at M = 1: 10.5 us streaming, 12.9 us through expansion + GEMM).
static bool w4_streaming_preferred(int M, int K) { return M <= W8_GEMV_PREFERRED_MAX_M && gemv_w8_fits(M, K); }

size_t bitrl_w8a8_workspace_bytes(int32_t M, int32_t K) {
  if (M < 1 || K < 1) return 0;
  if (w8_streaming_preferred(M, K)) return 0;
  return align_up(static_cast<size_t>(M) * K, 256) + align_up(static_cast<size_t>(M) * 4, 256);
}

static bitrl_status w8a8_impl(const int8_t* wq, const float* scale, const void* x, int32_t M, int32_t K, int32_t N, void* y,
                              int32_t out_dtype, void* workspace, size_t workspace_bytes, int8_t* xq_out,
                              float* absmax_out, int32_t* acc_out, void* stream) {
  if (!wq || !scale || !x || !y) return BITRL_ERR_NULL;
  if (M < 1 || !shape_ok(N, K)) return BITRL_ERR_SHAPE;
  if (out_dtype != BITRL_OUT_F32 && out_dtype != BITRL_OUT_BF16) return BITRL_ERR_DTYPE;
  if (!aligned16(wq) || !aligned16(x) || !aligned16(y) || !aligned16(workspace)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (gemv_w8_fits(M, K) &&
      (w8_streaming_preferred(M, K) || !workspace || workspace_bytes < bitrl_w8a8_workspace_bytes(M, K)))
    return launch_gemv_w8(wq, scale, N, K, x, M, y, out_dtype, xq_out, absmax_out, acc_out, st);
  if (!workspace || workspace_bytes < bitrl_w8a8_workspace_bytes(M, K)) return BITRL_ERR_WORKSPACE;
  int8_t* xq = static_cast<int8_t*>(workspace);
  float* absmax = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + align_up(static_cast<size_t>(M) * K, 256));
  if ((s = launch_quant_act(x, M, K, xq, absmax, nullptr, st)) != BITRL_OK) return s;
  if ((s = launch_gemm_w8(wq, scale, N, K, xq, absmax, M, y, out_dtype, nullptr, acc_out, st)) != BITRL_OK) return s;
  if (xq_out) BITRL_CUDA(cudaMemcpyAsync(xq_out, xq, static_cast<size_t>(M) * K, cudaMemcpyDeviceToDevice, st));
  if (absmax_out) BITRL_CUDA(cudaMemcpyAsync(absmax_out, absmax, static_cast<size_t>(M) * 4, cudaMemcpyDeviceToDevice, st));
  return BITRL_OK;
}

bitrl_status bitrl_w8a8_forward(const int8_t* wq, const float* scale, const void* x, int32_t M, int32_t K, int32_t N,
                                void* y, int32_t out_dtype, void* workspace, size_t workspace_bytes, void* stream) {
  return w8a8_impl(wq, scale, x, M, K, N, y, out_dtype, workspace, workspace_bytes, nullptr, nullptr, nullptr, stream);
}

bitrl_status bitrl_w8a8_forward_debug(const int8_t* wq, const float* scale, const void* x, int32_t M, int32_t K, int32_t N,
                                      void* y, int32_t out_dtype, void* workspace, size_t workspace_bytes, int8_t* xq_out,
                                      float* absmax_out, int32_t* acc_out, void* stream) {
  return w8a8_impl(wq, scale, x, M, K, N, y, out_dtype, workspace, workspace_bytes, xq_out, absmax_out, acc_out, stream);
}

bitrl_status bitrl_w8a8_forward_multi(int32_t count, const bitrl_w8_matrix_t* mats, const void* const* x, void* const* y,
                                      int32_t M, int32_t out_dtype, void* stream) {
  if (!mats || !x || !y) return BITRL_ERR_NULL;
  if (count < 1 || count > BITRL_MULTI_MAX_JOBS || M < 1 || M > BITRL_W8_MULTI_MAX_M) return BITRL_ERR_SHAPE;
  if (out_dtype != BITRL_OUT_F32 && out_dtype != BITRL_OUT_BF16) return BITRL_ERR_DTYPE;
  W8Matrix w[BITRL_MULTI_MAX_JOBS];
  for (int i = 0; i < count; ++i) {
    if (!mats[i].wq || !mats[i].scale || !x[i] || !y[i]) return BITRL_ERR_NULL;
    if (!shape_ok(mats[i].N, mats[i].K) || mats[i].K > 32768) return BITRL_ERR_SHAPE;
    if (!aligned16(mats[i].wq) || !aligned16(x[i]) || !aligned16(y[i])) return BITRL_ERR_ALIGN;
    w[i] = W8Matrix{mats[i].wq, mats[i].scale, mats[i].N, mats[i].K};
  }
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_gemv8_multi(count, w, x, y, M, out_dtype, false, static_cast<cudaStream_t>(stream));
}

// ---- W4A8 layer (INT4 critic) -----------------------------------------------------------------------------------

bitrl_status bitrl_w4_quantize(const float* W, int32_t N, int32_t K, uint8_t* packed, float* scale, void* stream) {
  if (!W || !packed || !scale) return BITRL_ERR_NULL;
  if (!shape_ok(N, K)) return BITRL_ERR_SHAPE;
  if (!aligned16(W) || !aligned16(packed)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_w4_quantize(W, N, K, packed, scale, static_cast<cudaStream_t>(stream));
}

size_t bitrl_w4a8_workspace_bytes(int32_t M, int32_t K, int32_t N) {
  if (M < 1 || K < 1 || N < 1) return 0;
  if (w4_streaming_preferred(M, K)) return 0;
  return bitrl_w8a8_workspace_bytes(M, K) + align_up(static_cast<size_t>(N) * K, 256);
}

static bitrl_status w4a8_impl(const uint8_t* packed, const float* scale, const void* x, int32_t M, int32_t K, int32_t N,
                              void* y, int32_t out_dtype, void* workspace, size_t workspace_bytes, int8_t* xq_out,
                              float* absmax_out, int32_t* acc_out, void* stream) {
  if (!packed || !scale || !x || !y) return BITRL_ERR_NULL;
  if (M < 1 || !shape_ok(N, K)) return BITRL_ERR_SHAPE;
  if (out_dtype != BITRL_OUT_F32 && out_dtype != BITRL_OUT_BF16) return BITRL_ERR_DTYPE;
  if (!aligned16(packed) || !aligned16(x) || !aligned16(y) || !aligned16(workspace)) return BITRL_ERR_ALIGN;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (gemv_w8_fits(M, K) &&
      (w4_streaming_preferred(M, K) || !workspace || workspace_bytes < bitrl_w4a8_workspace_bytes(M, K, N)))
    return launch_gemv_w4(packed, scale, N, K, x, M, y, out_dtype, xq_out, absmax_out, acc_out, st);
  if (!workspace || workspace_bytes < bitrl_w4a8_workspace_bytes(M, K, N)) return BITRL_ERR_WORKSPACE;
  unsigned char* b = static_cast<unsigned char*>(workspace);
  int8_t* xq = reinterpret_cast<int8_t*>(b);
  float* absmax = reinterpret_cast<float*>(b + align_up(static_cast<size_t>(M) * K, 256));
  int8_t* w8 = reinterpret_cast<int8_t*>(b + bitrl_w8a8_workspace_bytes(M, K));
  if ((s = launch_quant_act(x, M, K, xq, absmax, nullptr, st)) != BITRL_OK) return s;
  if ((s = launch_w4_expand(packed, N, K, w8, st)) != BITRL_OK) return s;
  if ((s = launch_gemm_w8(w8, scale, N, K, xq, absmax, M, y, out_dtype, nullptr, acc_out, st)) != BITRL_OK) return s;
  if (xq_out) BITRL_CUDA(cudaMemcpyAsync(xq_out, xq, static_cast<size_t>(M) * K, cudaMemcpyDeviceToDevice, st));
  if (absmax_out) BITRL_CUDA(cudaMemcpyAsync(absmax_out, absmax, static_cast<size_t>(M) * 4, cudaMemcpyDeviceToDevice, st));
  return BITRL_OK;
}

bitrl_status bitrl_w4a8_forward(const uint8_t* packed, const float* scale, const void* x, int32_t M, int32_t K, int32_t N,
                                void* y, int32_t out_dtype, void* workspace, size_t workspace_bytes, void* stream) {
  return w4a8_impl(packed, scale, x, M, K, N, y, out_dtype, workspace, workspace_bytes, nullptr, nullptr, nullptr, stream);
}

bitrl_status bitrl_w4a8_forward_debug(const uint8_t* packed, const float* scale, const void* x, int32_t M, int32_t K,
                                      int32_t N, void* y, int32_t out_dtype, void* workspace, size_t workspace_bytes,
                                      int8_t* xq_out, float* absmax_out, int32_t* acc_out, void* stream) {
  return w4a8_impl(packed, scale, x, M, K, N, y, out_dtype, workspace, workspace_bytes, xq_out, absmax_out, acc_out, stream);
}

// ---- five weights per byte: the denser format of the streaming path ---------------------------------------------

bitrl_status bitrl_pack5(const uint8_t* packed, int32_t N, int32_t K, uint8_t* packed5, void* stream) {
  if (!packed || !packed5) return BITRL_ERR_NULL;
  if (!shape_ok(N, K)) return BITRL_ERR_SHAPE;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  const long long n = static_cast<long long>(N) * ((K + 4) / 5);
  pack5_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(packed, N, K, packed5);
  count_launch(1);
  BITRL_CUDA(cudaGetLastError());
  return BITRL_OK;
}

bitrl_status bitrl_linear5_create(const uint8_t* packed5, const float* gamma, int32_t N, int32_t K,
                                  bitrl_linear5_t** out, void* stream) {
  if (!packed5 || !gamma || !out) return BITRL_ERR_NULL;
  if (!shape_ok(N, K)) return BITRL_ERR_SHAPE;
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  bitrl_linear5* w = new (std::nothrow) bitrl_linear5();
  if (!w) return BITRL_ERR_CUDA;
  w->l = Linear5{nullptr, nullptr, N, K, (K + T5_K - 1) / T5_K};
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = static_cast<size_t>(N / TILE_ROWS) * w->l.pieces * TILE_BYTES;
  cudaError_t e = cudaMalloc(&w->l.tiles, bytes);
  if (e == cudaSuccess) e = cudaMalloc(&w->l.gamma, 256);
  if (e == cudaSuccess) e = cudaMemcpyAsync(w->l.gamma, gamma, sizeof(float), cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess) {
    retile5_kernel<<<static_cast<unsigned>((bytes + 255) / 256), 256, 0, st>>>(packed5, N, K, w->l.pieces, w->l.tiles);
    count_launch(1);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);  // the handle is complete when this returns
  if (e != cudaSuccess) {
    cudaFree(w->l.tiles);
    cudaFree(w->l.gamma);
    delete w;
    return cuda_fail(e);
  }
  *out = w;
  return BITRL_OK;
}

bitrl_status bitrl_linear5_destroy(bitrl_linear5_t* w) {
  if (!w) return BITRL_OK;
  cudaFree(w->l.tiles);
  cudaFree(w->l.gamma);
  delete w;
  return BITRL_OK;
}

size_t bitrl_linear5_bytes(const bitrl_linear5_t* w) {
  return w ? static_cast<size_t>(w->l.N / TILE_ROWS) * w->l.pieces * TILE_BYTES : 0;
}

bitrl_status bitrl_bitlinear5_forward_multi(int32_t count, const bitrl_linear5_t* const* w, const void* const* x,
                                            void* const* y, int32_t M, int32_t out_dtype, void* stream) {
  if (!w || !x || !y) return BITRL_ERR_NULL;
  if (count < 1 || count > BITRL_MULTI_MAX_JOBS || M < 1 || M > BITRL_LINEAR5_MAX_M) return BITRL_ERR_SHAPE;
  if (out_dtype != BITRL_OUT_F32 && out_dtype != BITRL_OUT_BF16) return BITRL_ERR_DTYPE;
  const Linear5* lins[BITRL_MULTI_MAX_JOBS];
  for (int i = 0; i < count; ++i) {
    if (!w[i] || !x[i] || !y[i]) return BITRL_ERR_NULL;
    if (!aligned16(x[i]) || !aligned16(y[i])) return BITRL_ERR_ALIGN;
    lins[i] = &w[i]->l;
  }
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_gemv5_multi(count, lins, x, y, M, out_dtype, static_cast<cudaStream_t>(stream));
}

bitrl_status bitrl_w4a8_forward_multi(int32_t count, const bitrl_w4_matrix_t* mats, const void* const* x, void* const* y,
                                      int32_t M, int32_t out_dtype, void* stream) {
  if (!mats || !x || !y) return BITRL_ERR_NULL;
  if (count < 1 || count > BITRL_MULTI_MAX_JOBS || M < 1 || M > BITRL_W8_MULTI_MAX_M) return BITRL_ERR_SHAPE;
  if (out_dtype != BITRL_OUT_F32 && out_dtype != BITRL_OUT_BF16) return BITRL_ERR_DTYPE;
  W8Matrix w[BITRL_MULTI_MAX_JOBS];
  for (int i = 0; i < count; ++i) {
    if (!mats[i].packed || !mats[i].scale || !x[i] || !y[i]) return BITRL_ERR_NULL;
    if (!shape_ok(mats[i].N, mats[i].K) || mats[i].K > 32768) return BITRL_ERR_SHAPE;
    if (!aligned16(mats[i].packed) || !aligned16(x[i]) || !aligned16(y[i])) return BITRL_ERR_ALIGN;
    w[i] = W8Matrix{reinterpret_cast<const int8_t*>(mats[i].packed), mats[i].scale, mats[i].N, mats[i].K};
  }
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  return launch_gemv8_multi(count, w, x, y, M, out_dtype, true, static_cast<cudaStream_t>(stream));
}

// ---- self-test of the bounded-wait / status-word path ----
}  // extern "C"
namespace {
__global__ void selftest_wait_kernel(long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = ptx::smem_u32(&bar);
  ptx::mbar_init(b, 1);
  ptx::mbar_init_fence();
  if (!ptx::mbar_wait(b, 0, limit_cycles)) report_timeout(99);  // nobody arrives: the wait must give up
}
}  // namespace
extern "C" {

bitrl_status bitrl_selftest_wait_timeout(int64_t limit_cycles, void* stream) {
  bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  long long lim = limit_cycles < 1000 ? 1000 : (limit_cycles > 1000000000LL ? 1000000000LL : limit_cycles);
  selftest_wait_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(lim);
  count_launch(1);
  BITRL_CUDA(cudaGetLastError());
  return BITRL_OK;
}

// ---- status -------------------------------------------------------------------------------------------

bitrl_status bitrl_poll_status(void* stream) {
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e);
  int h[4] = {0, 0, 0, 0};
  e = cudaMemcpyFromSymbol(h, g_status, sizeof(h));
  if (e != cudaSuccess) return cuda_fail(e);
  if (h[0] != 0) {
    g_last_stage.store(h[1]);
    const int z[4] = {0, 0, 0, 0};
    e = cudaMemcpyToSymbol(g_status, z, sizeof(z));
    if (e != cudaSuccess) return cuda_fail(e);
    return h[0];
  }
  return BITRL_OK;
}

int32_t bitrl_last_timeout_stage(void) { return g_last_stage.load(); }
int32_t bitrl_last_cuda_error(void) { return g_last_cuda.load(); }
uint64_t bitrl_launch_count(void) { return g_launches.load(); }

bitrl_status bitrl_gemm_plan(int32_t M, int32_t K, int32_t N, int32_t with_workspace, int32_t* tok, int32_t* splits,
                             int32_t* kind) {
  if (M < 1 || K < 128 || N < 128 || K % 128 != 0 || N % 128 != 0) return BITRL_ERR_SHAPE;
  const bitrl_status s = check_arch();
  if (s != BITRL_OK) return s;
  const GemmPlan p = gemm_plan(N, K, M, with_workspace != 0);
  if (tok) *tok = p.tok;
  if (splits) *splits = p.splits;
  if (kind)
    *kind = p.pair ? BITRL_GEMM_PAIRED
                   : p.splits == 1 ? BITRL_GEMM_SINGLE : p.clsk ? BITRL_GEMM_SPLIT_CLUSTER : BITRL_GEMM_SPLIT_SCRATCH;
  return BITRL_OK;
}

const char* bitrl_status_string(bitrl_status s) {
  switch (s) {
    case BITRL_OK: return "ok";
    case BITRL_ERR_NULL: return "null pointer";
    case BITRL_ERR_SHAPE: return "bad shape";
    case BITRL_ERR_ALIGN: return "pointer not 16-byte aligned";
    case BITRL_ERR_ARCH: return "device is not compute capability 10.0";
    case BITRL_ERR_CUDA: return "CUDA error";
    case BITRL_ERR_TIMEOUT: return "device-side wait timed out";
    case BITRL_ERR_WORKSPACE: return "workspace missing or too small";
    case BITRL_ERR_DTYPE: return "bad output dtype";
    case BITRL_ERR_LIMIT: return "size beyond the fixed maximum of this entry point";
    default: return "unknown status";
  }
}

}  // extern "C"
