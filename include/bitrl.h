/*
 * bitrl.h - C ABI of the BitLinear W1.58A8 hot path of the BitRL frozen backbone, for NVIDIA B200 (sm_100a).
 *
 * The layer (paper: Sec. III-A, Eq. 2 and the paragraph after Eq. 3; Sec. V, edge-deployment paragraph):
 *   weights are ternary {-1,0,+1}, Q(W) = sign(W) * 1[|W| > tau] (Eq. 2), inference is integer arithmetic
 *   without floating multiply-accumulate, ternary products being additions and subtractions.
 * The paper leaves tau, the activation format and the scales open; this library takes the W1.58A8 layer of the
 * BitNet b1.58 architecture the paper's backbone follows:
 *   gamma = mean|W| (per matrix),  W_q = clip(rint(W / (gamma + 1e-5)), -1, 1)     [= Eq. 2, tau = (gamma+1e-5)/2]
 *   a_m   = max(max_k |x[m,k]|, 1e-5),  x_q[m,k] = clip(rint(x[m,k] * (127 / a_m)), -128, 127)
 *   acc[m,n] = sum_k x_q[m,k] * W_q[n,k]                                   (int32, exact)
 *   y[m,n]   = (float)acc[m,n] * (gamma * (a_m / 127))                     (fp32, then bf16 RNE if asked)
 * rint is round-to-nearest, ties-to-even; each fp32 step is one IEEE operation in the order written.
 *
 * Conventions
 *   - Every pointer marked "dev" is device memory on the current CUDA device; "host" is host memory.
 *   - Matrices are row-major.  W is [N, K] (out x in), x is [M, K], y is [M, N]:  y = x * W^T.
 *   - K and N must be multiples of 128; device pointers must be 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Calls are asynchronous on `stream`.  Argument errors are returned at once; a device-side wait that gave
 *     up (every wait in the kernels is bounded) is reported by bitrl_poll_status.
 *   - The caller owns every buffer it passes, including workspaces.  The library owns what *_create returns.
 *   - No entry point allocates device memory except the *_create functions.  Nothing throws, aborts or traps.
 */
#ifndef BITRL_H_
#define BITRL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define BITRL_API __attribute__((visibility("default")))
#else
#define BITRL_API
#endif

typedef int32_t bitrl_status;
#define BITRL_OK 0
#define BITRL_ERR_NULL (-1)      /* a required pointer is NULL */
#define BITRL_ERR_SHAPE (-2)     /* M < 1, K or N not a multiple of 128, shape does not match the handle, bad state offsets */
#define BITRL_ERR_ALIGN (-3)     /* a device pointer is not 16-byte aligned */
#define BITRL_ERR_ARCH (-4)      /* current device is not compute capability 10.0 */
#define BITRL_ERR_CUDA (-5)      /* a CUDA call failed; code in bitrl_last_cuda_error() */
#define BITRL_ERR_TIMEOUT (-6)   /* a bounded device-side wait expired (see bitrl_poll_status) */
#define BITRL_ERR_WORKSPACE (-7) /* workspace missing or smaller than the *_workspace_bytes query */
#define BITRL_ERR_DTYPE (-8)     /* unknown out_dtype */
#define BITRL_ERR_LIMIT (-9)     /* size beyond the fixed maximum of an entry point that cannot allocate */

#define BITRL_OUT_F32 0
#define BITRL_OUT_BF16 1

/* Largest M served by the streaming (GEMV) kernel; larger M runs the tcgen05 GEMM kernel. */
#define BITRL_GEMV_MAX_M 16

typedef struct bitrl_linear bitrl_linear_t;   /* packed ternary weights in kernel layout + gamma + N, K */
typedef struct bitrl_encoder bitrl_encoder_t; /* a stack of blocks of four bitrl_linear_t each */

/* ---- a0: ternarize + pack (offline, once per matrix; the backbone is frozen - Sec. III-A) ---------------
 * Eq. 2 with tau = (gamma+1e-5)/2.  W: dev fp32 [N,K].  packed: dev [N, K/4] bytes, canonical format:
 * code c = W_q + 1 in {0,1,2}; byte j of row n holds k = 4j..4j+3, code of k in bits [2(k%4)+1 : 2(k%4)].
 * gamma: dev fp32 [1].  |W| is summed in fp64 (fixed tree order, deterministic) and rounded once to fp32.
 * workspace: dev, at least bitrl_pack_workspace_bytes(N, K) bytes. */
BITRL_API size_t bitrl_pack_workspace_bytes(int32_t N, int32_t K);
BITRL_API bitrl_status bitrl_pack_ternary(const float* W, int32_t N, int32_t K, uint8_t* packed, float* gamma,
                                void* workspace, size_t workspace_bytes, void* stream);

/* Same result as bitrl_pack_ternary, for callers that have no device memory to spare for a workspace and are not
 * allowed to obtain any: code that runs inside a memory pool it must not grow, inside a stream-ordered region
 * where cudaMalloc would serialize the device, or in a process whose allocator is owned by another framework.
 * (The paper has no counterpart; this is a convenience of this library.)  The fp64 partial sums of |W| live in a
 * fixed 8 KB array that is part of the library image on every GPU that loads it, for the life of the process.
 *  - Limit: N*K <= BITRL_PACK_STATIC_MAX_WEIGHTS; larger matrices return BITRL_ERR_LIMIT and nothing is launched.
 *  - Calls no allocator of any kind.  The first call on a device looks up the array's device address (once per
 *    device, with that device current); make that first call outside any stream capture.  The address is kept for
 *    the life of the device's context: after cudaDeviceReset the library must be reloaded before this call is used again.
 *  - All calls share the array and it keeps the previous call's contents.  Nothing in it has to start at zero:
 *    every slot that a call reads is written earlier in the same call.  Two calls that overlap on the GPU (different
 *    streams, or threads) race on it and may both produce a wrong gamma; serialize them. */
#define BITRL_PACK_STATIC_MAX_WEIGHTS (1LL << 28)
BITRL_API bitrl_status bitrl_pack_ternary_static(const float* W, int32_t N, int32_t K, uint8_t* packed, float* gamma,
                                                 void* stream);

/* Builds the weight handle from the canonical packed bytes and gamma (both dev).  The library keeps its own
 * re-tiled copy (N*K/4 bytes).  The call returns after the copy is complete (it synchronizes `stream`: handle creation
 * is offline work and already allocates), so the inputs may be freed at once and the handle may be used on any stream.
 * The forward kernels treat a handle's weights as immutable and fetch them before they wait for preceding kernels. */
BITRL_API bitrl_status bitrl_linear_create(const uint8_t* packed, const float* gamma, int32_t N, int32_t K,
                                 bitrl_linear_t** out, void* stream);
BITRL_API bitrl_status bitrl_linear_destroy(bitrl_linear_t* w);

/* ---- a1: per-token absmax int8 activation quantization (Q = 127) ---------------------------------------
 * x: dev bf16 [M,K].  xq: dev int8 [M,K].  absmax: dev fp32 [M] (the clamped a_m).
 * rowsum: dev int32 [M] = sum_k x_q[m,k], or NULL.  (The GEMM feeds weight codes W_q+1 as unsigned bytes
 * and repays sum_k x_q once per output; the row sum is that correction.) */
BITRL_API bitrl_status bitrl_quant_act(const void* x, int32_t M, int32_t K, int8_t* xq, float* absmax, int32_t* rowsum,
                             void* stream);

/* ---- a1..a3: the whole layer  y = BitLinear(x) --------------------------------------------------------
 * x: dev bf16 [M,K]; y: dev [M,N] fp32 (BITRL_OUT_F32) or bf16 (BITRL_OUT_BF16).  K, N must equal the
 * handle's.  M <= 4: one streaming kernel (quantization in its prologue, rescale in its epilogue; no workspace
 * needed).  Larger M: quantization kernel into the workspace, then the tcgen05 GEMM.  For 5 <= M <= BITRL_GEMV_MAX_M
 * the workspace is optional: without it (NULL, or too small) the streaming kernel serves the call, 1.4-3 x slower.
 * workspace: dev, >= bitrl_workspace_bytes(M,K,N) (0 for M <= 4, then NULL is accepted).  The results are the same
 * bits whichever kernel runs.
 * When a launch has too few output tiles to occupy the SMs, K is split across them.  Narrow token tiles (<= 128
 * tokens) do that inside one launch: the CTAs of a thread-block cluster take the k ranges of one tile and exchange
 * their exact int32 partial sums through distributed shared memory.  Otherwise, up to M = 512, the workspace also
 * holds M*N int32 of scratch where the partial sums meet (integer atomics: order-free, deterministic) and a
 * finishing kernel applies the rescale.  The results are the same bits in every form. */
BITRL_API size_t bitrl_workspace_bytes(int32_t M, int32_t K, int32_t N);
/* Which kernel form the launcher takes for an [M,K] x [N,K]^T product with M > BITRL_GEMV_MAX_M on the current device
 * (a query for tests and diagnostics; launches nothing).  tok: tokens per tile (64 ... 256).  splits: k ranges per tile.
 * kind: BITRL_GEMM_SINGLE (one CTA per tile, splits = 1), BITRL_GEMM_SPLIT_SCRATCH, BITRL_GEMM_SPLIT_CLUSTER or
 * BITRL_GEMM_PAIRED (256-row tiles on CTA pairs).  with_workspace != 0: the caller would pass the workspace above.
 * Any of the three output pointers may be NULL.  BITRL_ERR_SHAPE unless N, K are multiples of 128 and M >= 1. */
#define BITRL_GEMM_SINGLE 0
#define BITRL_GEMM_SPLIT_SCRATCH 1
#define BITRL_GEMM_SPLIT_CLUSTER 2
#define BITRL_GEMM_PAIRED 3
BITRL_API bitrl_status bitrl_gemm_plan(int32_t M, int32_t K, int32_t N, int32_t with_workspace, int32_t* tok,
                                       int32_t* splits, int32_t* kind);
BITRL_API bitrl_status bitrl_bitlinear_forward(const bitrl_linear_t* w, const void* x, int32_t M, int32_t K, int32_t N,
                                     void* y, int32_t out_dtype, void* workspace, size_t workspace_bytes,
                                     void* stream);

/* `count` independent layers in one launch, for M <= BITRL_GEMV_MAX_M: y[i] = BitLinear_{w[i]}(x[i]).  One decode-size
 * matrix is only a few MB, so a launch per matrix is bound by launch latency; when the calls do not depend on one
 * another (a sweep over matrices, several projections of the same input) this entry point streams all their packed
 * weights back to back at HBM speed with one persistent kernel.  w, x, y: HOST arrays of `count` entries; x[i] dev
 * bf16 [M, K_i] (entries may repeat), y[i] dev [M, N_i], all distinct.  1 <= count <= BITRL_MULTI_MAX_JOBS.  No workspace.
 * Results are bit-identical to `count` separate bitrl_bitlinear_forward calls. */
#define BITRL_MULTI_MAX_JOBS 128
BITRL_API bitrl_status bitrl_bitlinear_forward_multi(int32_t count, const bitrl_linear_t* const* w,
                                                     const void* const* x, void* const* y, int32_t M,
                                                     int32_t out_dtype, void* stream);

/* Same, and additionally writes the integer stages: xq_out dev int8 [M,K], absmax_out dev fp32 [M],
 * acc_out dev int32 [M,N] (any may be NULL).  Needs the workspace for every M. */
BITRL_API bitrl_status bitrl_bitlinear_forward_debug(const bitrl_linear_t* w, const void* x, int32_t M, int32_t K,
                                           int32_t N, void* y, int32_t out_dtype, void* workspace,
                                           size_t workspace_bytes, int8_t* xq_out, float* absmax_out,
                                           int32_t* acc_out, void* stream);

/* a2 + a3 on an already quantized input (what a fused producer hands over).
 * xq dev int8 [M,K], absmax dev fp32 [M], rowsum dev int32 [M] (all required).
 * residual: NULL, or dev bf16 [M,N]; then y = bf16( fp32(residual) + fp32(bf16(acc*scale)) ), out_dtype must be
 * BITRL_OUT_BF16, and y may alias residual.  acc_out: NULL or dev int32 [M,N]. */
BITRL_API bitrl_status bitrl_bitlinear_forward_q(const bitrl_linear_t* w, const int8_t* xq, const float* absmax,
                                       const int32_t* rowsum, int32_t M, void* y, int32_t out_dtype,
                                       const void* residual, int32_t* acc_out, void* stream);

/* ---- a4: fused producers of the encoder block (the architecture is cited, not spelled out, by the paper:
 * Sec. III-B takes the backbone architecture from the BitNet papers by reference; gain 1, eps 1e-5) -------
 * Each computes u = bf16( v / sqrt(mean_k v^2 + 1e-5) ) in fp32 for its row vector v and then quantizes u
 * exactly like bitrl_quant_act.  u_out: NULL or dev bf16 [T, K_out] (the value that was quantized).
 *   rmsnorm_quant:            v = h[t, :]                                   h: dev bf16 [T,K]
 *   vrepeat_rmsnorm_quant:    v = V of qkv[t], each kv head repeated n_heads/n_kv_heads times ("identity
 *                             attention": one key per query, so softmax = 1)  qkv: dev bf16 [T,(n_heads+2 n_kv)*hd]
 *   relu2gate_rmsnorm_quant:  v = max(g,0)^2 * up, gu = [g | up]              gu: dev bf16 [T, 2F] */
BITRL_API bitrl_status bitrl_rmsnorm_quant(const void* h, int32_t T, int32_t K, int8_t* xq, float* absmax,
                                 int32_t* rowsum, void* u_out, void* stream);
BITRL_API bitrl_status bitrl_vrepeat_rmsnorm_quant(const void* qkv, int32_t T, int32_t n_heads, int32_t n_kv_heads,
                                         int32_t head_dim, int8_t* xq, float* absmax, int32_t* rowsum,
                                         void* u_out, void* stream);
BITRL_API bitrl_status bitrl_relu2gate_rmsnorm_quant(const void* gu, int32_t T, int32_t F, int8_t* xq, float* absmax,
                                           int32_t* rowsum, void* u_out, void* stream);

/* ---- frozen encoder f_theta* (Eq. 3): L blocks of {qkv, out, gate/up, down} ----------------------------
 * layers: host array of 4*L handles ordered qkv, out, gateup, down per block; the handles must outlive the
 * encoder.  d = n_heads*head_dim; qkv has N = d + 2*n_kv_heads*head_dim, gateup N = 2*d_ff, down K = d_ff.
 * Block:  h += out(RMSNorm(repeat(V(qkv(RMSNorm(h))))));  h += down(RMSNorm(relu(g)^2 * up)), [g|up] = gateup(RMSNorm(h)).
 * h_in, h_out: dev bf16 [T,d] (may alias).  workspace >= bitrl_encoder_workspace_bytes(enc, T). */
BITRL_API bitrl_status bitrl_encoder_create(const bitrl_linear_t* const* layers, int32_t L, int32_t d, int32_t d_ff,
                                  int32_t n_heads, int32_t n_kv_heads, bitrl_encoder_t** enc);
BITRL_API bitrl_status bitrl_encoder_destroy(bitrl_encoder_t* enc);
BITRL_API size_t bitrl_encoder_workspace_bytes(const bitrl_encoder_t* enc, int32_t T);
BITRL_API bitrl_status bitrl_encoder_forward(const bitrl_encoder_t* enc, const void* h_in, int32_t T, void* h_out,
                                   void* workspace, size_t workspace_bytes, void* stream);

/* ---- attention inside each state (the step of the encoder block that the contraction feeds; Eq. 3 encodes every
 * state s_t on its own, Sec. V: 15-40 tokens per state, one forward pass) --------------------------------------
 * Causal grouped-query attention with rotary position embedding (rotate-half form) over independent states:
 *   angle(p, i) = p * theta^(-2i/head_dim), p = index of the token inside its state, i < head_dim/2
 *   (x_i, x_{i+hd/2}) -> (x_i cos - x_{i+hd/2} sin, x_{i+hd/2} cos + x_i sin)          applied to q and k
 *   att[p] = sum_{r<=p} softmax_r(q_p . k_r / sqrt(head_dim)) v_r ; query head h reads kv head h / (n_heads/n_kv_heads)
 * fp32 arithmetic, cos/sin from an fp64 table, one rounding to bf16.
 * qkv: dev bf16 [T, (n_heads + 2 n_kv_heads) * head_dim] = [q | k | v].  att: dev bf16 [T, n_heads * head_dim].
 * States: state_off = dev int32 [n_states + 1], ascending token offsets with state_off[0] = 0 and
 * state_off[n_states] = T, every length in 1..max_state_len; or NULL, then every state has max_state_len tokens and
 * T = n_states * max_state_len.  max_state_len <= BITRL_ATTN_MAX_STATE_TOKENS; head_dim is 64 or 128.
 * Offsets are read on the device: a state that breaks the rules above is skipped (its rows of att are not written)
 * and the next bitrl_poll_status returns BITRL_ERR_SHAPE.
 * workspace: dev, >= bitrl_attention_workspace_bytes(max_state_len, head_dim) (the rotary table). */
#define BITRL_ATTN_MAX_STATE_TOKENS 128
BITRL_API size_t bitrl_attention_workspace_bytes(int32_t max_state_len, int32_t head_dim);
BITRL_API bitrl_status bitrl_attention(const void* qkv, int32_t T, const int32_t* state_off, int32_t n_states,
                                       int32_t max_state_len, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                                       double theta, void* att, void* workspace, size_t workspace_bytes, void* stream);

/* Last-token pooling: out[s, :] = h[last token of state s, :], the latent h_t of Eq. 3 (one per state).
 * h: dev bf16 [T, d]; out: dev bf16 [n_states, d]; d a multiple of 8; states as for bitrl_attention. */
BITRL_API bitrl_status bitrl_pool_last_token(const void* h, int32_t T, const int32_t* state_off, int32_t n_states,
                                             int32_t max_state_len, int32_t d, void* out, void* stream);

/* The encoder with real attention in place of the identity on V:
 *   h += out(RMSNorm(attention(qkv(RMSNorm(h)))));  h += down(RMSNorm(relu(g)^2 * up))      per block,
 * states and theta as for bitrl_attention.  pooled: NULL, or dev bf16 [n_states, d] that receives the last token
 * of every state after the last block.  workspace >= bitrl_encoder_states_workspace_bytes(enc, T, max_state_len). */
BITRL_API size_t bitrl_encoder_states_workspace_bytes(const bitrl_encoder_t* enc, int32_t T, int32_t max_state_len);
BITRL_API bitrl_status bitrl_encoder_forward_states(const bitrl_encoder_t* enc, const void* h_in, int32_t T,
                                                    const int32_t* state_off, int32_t n_states, int32_t max_state_len,
                                                    double theta, void* h_out, void* pooled, void* workspace,
                                                    size_t workspace_bytes, void* stream);

/* ---- after the encoder: trainable heads, advantage estimation, PPO objective (all fp32, batched over the parallel
 * environments; Eq. 3, Eq. 1, Sec. III-B, Table VI) -----------------------------------------------------------
 * Heads: out = tanh(tanh(h W1t + b1) W2t + b2) W3t + b3.  The paper fixes two hidden layers of 256 and 128 units in
 * fp32 and gives no activation; tanh is used.  h: dev bf16 [B,d] (the pooled latents), d a multiple of 16.
 * Weights are dev fp32, stored input-major: W1t [d,H1], W2t [H1,H2], W3t [H2,n_out]; H1, H2, n_out <= 256.
 * heads: HOST array of n_heads (<= 4) descriptors (policy head: n_out = number of actions; value head: n_out = 1);
 * out: HOST array of n_heads dev fp32 pointers, out[i] is [B, heads[i].n_out]. */
typedef struct bitrl_head {
  const float* W1t; const float* b1;
  const float* W2t; const float* b2;
  const float* W3t; const float* b3;
  int32_t n_out;
} bitrl_head_t;
BITRL_API bitrl_status bitrl_heads_forward(const void* h, int32_t B, int32_t d, int32_t H1, int32_t H2,
                                           const bitrl_head_t* heads, int32_t n_heads, float* const* out, void* stream);

/* Generalized advantage estimation over T steps of E environments (time-major dev fp32 arrays):
 *   delta_t = r_t + gamma V_{t+1} (1 - done_t) - V_t ;  A_t = delta_t + gamma lambda (1 - done_t) A_{t+1}, A_T = 0
 * rewards, dones: [T,E]; values: [T+1,E] (row T is the bootstrap value); adv: [T,E]; returns: NULL or [T,E] = adv + V. */
BITRL_API bitrl_status bitrl_gae(const float* rewards, const float* values, const float* dones, int32_t T, int32_t E,
                                 float gamma, float lambda, float* adv, float* returns, void* stream);

/* Clipped surrogate of Eq. 1 with entropy bonus, and the value error, over a batch of B samples with A actions:
 *   r = exp(log pi(a|s) - old_logp);  L_clip = mean min(r Ahat, clip(r, 1-eps, 1+eps) Ahat);  H = mean entropy(pi)
 *   policy_loss = -(L_clip + beta H);  value_loss = mean 0.5 (V - R)^2
 * logits: dev fp32 [B,A]; actions: dev int32 [B]; old_logp, adv, values, returns: dev fp32 [B].
 * terms: dev fp32 [B,4] = per sample {r, min(...), entropy, 0.5 (V-R)^2} (required; also the reduction's input).
 * dlogits: NULL or dev fp32 [B,A] = d policy_loss / d logits; dvalues: NULL or dev fp32 [B] = d value_loss / d values.
 * summary: dev fp32 [4] = {L_clip, H, policy_loss, value_loss}, summed in a fixed order (deterministic). */
BITRL_API bitrl_status bitrl_ppo_loss(const float* logits, const int32_t* actions, const float* old_logp,
                                      const float* adv, const float* values, const float* returns, int32_t B, int32_t A,
                                      float eps, float beta, float* terms, float* dlogits, float* dvalues,
                                      float* summary, void* stream);

/* ---- W8A8 layer: the higher-precision critic backbone (Sec. V ablations, Table IV: "INT8 critic + 1-bit policy";
 * the paper names the precision only) -------------------------------------------------------------------------
 * One symmetric absmax scale per matrix, rounding as for the activations:
 *   a = max(max|W|, 1e-20),  W_q = clip(rint(W * (127 / a)), -128, 127),  scale = a / 127
 *   acc[m,n] = sum_k x_q[m,k] * W_q[n,k] (int32),  y[m,n] = (float)acc[m,n] * (scale * (a_m / 127))
 * with x_q, a_m exactly as in bitrl_quant_act.  |acc| can exceed 2^24, so (float)acc is the int32 -> fp32 conversion
 * with round-to-nearest-even.
 * bitrl_w8_quantize: W dev fp32 [N,K] -> wq dev int8 [N,K] (row-major, the format the forward call reads) and
 * scale: dev fp32 [2] - scale[0] receives the scale, scale[1] is scratch of the call.
 * bitrl_w8a8_forward: x dev bf16 [M,K], y dev [M,N] fp32 or bf16.  M <= 4 and K <= 4096: one streaming kernel
 * (quantization in its prologue, dp4a, no workspace); otherwise: quantization kernel, then a tcgen05 GEMM with both
 * operands straight from TMA tiles (split over the CTAs of a cluster along K when the tiles are few).
 * workspace: dev, >= bitrl_w8a8_workspace_bytes(M, K) (0 where the streaming kernel is preferred, NULL accepted).  For
 * every M <= BITRL_GEMV_MAX_M the workspace is optional: without it (NULL or too small) the streaming kernel serves the
 * call, 1.2-3 x slower where it is not the preferred form.  Same bits either way.
 * The _debug variant also writes xq_out dev int8 [M,K], absmax_out dev fp32 [M], acc_out dev int32 [M,N] (any may be NULL). */
BITRL_API bitrl_status bitrl_w8_quantize(const float* W, int32_t N, int32_t K, int8_t* wq, float* scale, void* stream);
BITRL_API size_t bitrl_w8a8_workspace_bytes(int32_t M, int32_t K);
BITRL_API bitrl_status bitrl_w8a8_forward(const int8_t* wq, const float* scale, const void* x, int32_t M, int32_t K,
                                          int32_t N, void* y, int32_t out_dtype, void* workspace, size_t workspace_bytes,
                                          void* stream);
BITRL_API bitrl_status bitrl_w8a8_forward_debug(const int8_t* wq, const float* scale, const void* x, int32_t M, int32_t K,
                                                int32_t N, void* y, int32_t out_dtype, void* workspace,
                                                size_t workspace_bytes, int8_t* xq_out, float* absmax_out,
                                                int32_t* acc_out, void* stream);

/* `count` independent W8A8 layers in one launch, for M <= BITRL_W8_MULTI_MAX_M tokens (one state per step through a critic
 * backbone is a sweep over many decode-size matrices; a launch per matrix spends a third of its time ramping up):
 * y[i] = W8A8_{mats[i]}(x[i]), bit-identical to `count` bitrl_w8a8_forward calls.  mats, x, y: HOST arrays of `count`
 * entries (1 <= count <= BITRL_MULTI_MAX_JOBS); mats[i].wq dev int8 [N,K] row-major, mats[i].scale dev fp32 (the
 * scale), M * K <= 27648 (six 32 KB slots and the quantized activations share the SM's shared memory; else BITRL_ERR_SHAPE);
 * x[i] dev bf16 [M,K] (entries may repeat), y[i] dev [M,N], all distinct.  No workspace. */
#define BITRL_W8_MULTI_MAX_M 2
typedef struct bitrl_w8_matrix {
  const int8_t* wq;
  const float* scale;
  int32_t N, K;
} bitrl_w8_matrix_t;
BITRL_API bitrl_status bitrl_w8a8_forward_multi(int32_t count, const bitrl_w8_matrix_t* mats, const void* const* x,
                                                void* const* y, int32_t M, int32_t out_dtype, void* stream);

/* ---- W4A8 layer: the "INT4 critic" of the same table (the paper names the precision only) -------------------------
 * Same reading with 7 in place of 127:  a = max(max|W|, 1e-20),  W_q = clip(rint(W * (7 / a)), -8, 7),  scale = a / 7,
 * acc and y as for W8A8.  packed: dev uint8 [N, K/2], byte j of row n = (W_q[n,2j] + 8) | (W_q[n,2j+1] + 8) << 4.
 * bitrl_w4_quantize: W dev fp32 [N,K] -> packed and scale (dev fp32 [2]: scale[0] the result, scale[1] scratch).
 * bitrl_w4a8_forward: M <= 4 streams the packed bytes once (dp4a; no workspace); larger M expands the codes to int8 in
 * the workspace and runs the W8A8 GEMM on them.  workspace >= bitrl_w4a8_workspace_bytes(M, K, N) (0 for M <= 4); for
 * 5 <= M <= BITRL_GEMV_MAX_M it is optional, as for bitrl_w8a8_forward. */
BITRL_API bitrl_status bitrl_w4_quantize(const float* W, int32_t N, int32_t K, uint8_t* packed, float* scale, void* stream);
BITRL_API size_t bitrl_w4a8_workspace_bytes(int32_t M, int32_t K, int32_t N);
BITRL_API bitrl_status bitrl_w4a8_forward(const uint8_t* packed, const float* scale, const void* x, int32_t M, int32_t K,
                                          int32_t N, void* y, int32_t out_dtype, void* workspace, size_t workspace_bytes,
                                          void* stream);
BITRL_API bitrl_status bitrl_w4a8_forward_debug(const uint8_t* packed, const float* scale, const void* x, int32_t M,
                                                int32_t K, int32_t N, void* y, int32_t out_dtype, void* workspace,
                                                size_t workspace_bytes, int8_t* xq_out, float* absmax_out,
                                                int32_t* acc_out, void* stream);

/* The grouped launch for W4A8 layers, as bitrl_w8a8_forward_multi (same limits; mats[i].packed dev uint8 [N,K/2]);
 * bit-identical to `count` bitrl_w4a8_forward calls. */
typedef struct bitrl_w4_matrix {
  const uint8_t* packed;
  const float* scale;
  int32_t N, K;
} bitrl_w4_matrix_t;
BITRL_API bitrl_status bitrl_w4a8_forward_multi(int32_t count, const bitrl_w4_matrix_t* mats, const void* const* x,
                                                void* const* y, int32_t M, int32_t out_dtype, void* stream);

/* ---- five weights per byte: the denser, lookup-table-decoded format of the streaming path (Abstract: 1.58-bit
 * weights; Sec. V, edge-deployment paragraph: ternary products as additions and subtractions "with lookup tables") ----
 * Format (the paper gives none): byte j of row n = sum_{i=0..4} (W_q[n,5j+i] + 1) * 3^i, ceil(K/5) bytes per row,
 * positions beyond K counted as zero weights; 1.6 bits per weight against 2.
 * bitrl_pack5: packed dev [N,K/4] canonical 2-bit codes (the output of bitrl_pack_ternary) -> packed5 dev
 * [N, ceil(K/5)] bytes.  bitrl_linear5_create re-tiles packed5 into the kernel's layout (library-owned copy; returns
 * when it is complete) and bitrl_linear5_bytes reports the size of that copy, the bytes a forward call streams.
 * bitrl_bitlinear5_forward_multi: `count` independent layers y[i] = BitLinear_{w[i]}(x[i]) in one launch, like
 * bitrl_bitlinear_forward_multi, for M <= BITRL_LINEAR5_MAX_M tokens; every byte is decoded through a 243-entry table in
 * shared memory.  Results are bit-identical to the 2-bit path.  w, x, y: HOST arrays of `count` entries. */
#define BITRL_LINEAR5_MAX_M 2
typedef struct bitrl_linear5 bitrl_linear5_t;
BITRL_API bitrl_status bitrl_pack5(const uint8_t* packed, int32_t N, int32_t K, uint8_t* packed5, void* stream);
BITRL_API bitrl_status bitrl_linear5_create(const uint8_t* packed5, const float* gamma, int32_t N, int32_t K,
                                            bitrl_linear5_t** out, void* stream);
BITRL_API bitrl_status bitrl_linear5_destroy(bitrl_linear5_t* w);
BITRL_API size_t bitrl_linear5_bytes(const bitrl_linear5_t* w);
BITRL_API bitrl_status bitrl_bitlinear5_forward_multi(int32_t count, const bitrl_linear5_t* const* w,
                                                      const void* const* x, void* const* y, int32_t M,
                                                      int32_t out_dtype, void* stream);

/* ---- status ----------------------------------------------------------------------------------------- */
/* Synchronizes `stream`, then reads and clears the device status word.  BITRL_OK, BITRL_ERR_TIMEOUT (a kernel
 * wait expired; results of that launch are invalid) or BITRL_ERR_CUDA. */
BITRL_API bitrl_status bitrl_poll_status(void* stream);
/* Self-test of the failure path: launches a one-thread kernel that waits (for at most `limit_cycles` SM cycles,
 * clamped to [1e3, 1e9]) on a barrier that nothing ever signals, so the bounded wait expires and records stage 99.
 * The next bitrl_poll_status returns BITRL_ERR_TIMEOUT; the context stays usable.  No GPU fault is involved. */
BITRL_API bitrl_status bitrl_selftest_wait_timeout(int64_t limit_cycles, void* stream);
/* After BITRL_ERR_TIMEOUT: which wait gave up (kernel-specific stage id), else 0. */
BITRL_API int32_t bitrl_last_timeout_stage(void);
BITRL_API int32_t bitrl_last_cuda_error(void);
BITRL_API const char* bitrl_status_string(bitrl_status s);
/* Number of kernels this library has launched since load (all streams). */
BITRL_API uint64_t bitrl_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* BITRL_H_ */
