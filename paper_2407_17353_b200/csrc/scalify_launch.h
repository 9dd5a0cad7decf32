// Host-side launcher interfaces between the C ABI layer and the kernel translation units.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "scalify.h"

struct CUtensorMap_st;

namespace scalify {

int make_byte_map(CUtensorMap_st* map, const void* ptr, uint64_t inner, uint64_t rows, uint64_t batch, uint64_t ld,
                  uint64_t bs, uint32_t box_inner, uint32_t box_rows);
int make_byte_map4(CUtensorMap_st* map, const void* ptr, uint64_t inner, uint64_t rows, uint64_t heads, uint64_t batch,
                   uint64_t ld, uint64_t hs, uint64_t bs, uint32_t box_inner, uint32_t box_rows);

enum { kModeCast = 0, kModeDynamic = 1, kModeSet = 2 };

int64_t statistic_blocks_wanted(int64_t n, int elem_bytes);
int launch_statistic(const void* x, int dtype, int64_t n, int stat, void* ws, size_t ws_bytes, float* out_stat,
                     cudaStream_t st);
int launch_rescale_predicted(const void* x, int in_dt, void* y, int out_dt, int64_t n, int stat, const float* x_scale,
                             float* y_scale, void* ws, size_t ws_bytes, cudaStream_t st);
int launch_fused_rescale(const void* x, int in_dt, void* y, int out_dt, int64_t n, int stat, const float* x_scale,
                         float* y_scale, void* ws, size_t ws_bytes, cudaStream_t st);
int launch_rebalance(const void* x, int in_dt, void* y, int out_dt, int64_t n, const float* x_scale, float* y_scale,
                     const float* stat, const float* new_scale, int mode, uint32_t* status, cudaStream_t st);
int launch_rebalance_check(const void* x, int in_dt, void* y, int out_dt, int64_t n, const float* x_scale,
                            float* y_scale, const float* stat, const float* r_pred, float* hint_out,
                            uint32_t* status, cudaStream_t st);
int launch_scale_word_mul(float* scale, float c, cudaStream_t st);
int launch_add(const void* a, const void* b, int ab_dt, void* y, int out_dt, int64_t n, int64_t row_len, int broadcast,
               const float* a_scale, const float* b_scale, float* y_scale, int subtract, cudaStream_t st);
int launch_gelu(const void* x, const void* g, int in_dt, void* y, int out_dt, int64_t n, const float* x_scale,
                const float* g_scale, float* y_scale, int exact, int bwd, cudaStream_t st);
int launch_layernorm_fwd(const void* X, int x_dt, int64_t x_ld, void* Y, int y_dt, int64_t y_ld, int R, int d,
                         const void* gamma, const void* beta, int gb_dt, const float* gamma_scale,
                         const float* beta_scale, float* y_scale, float eps, int eps_inside, float* mean,
                         float* rinv, cudaStream_t st);
size_t layernorm_bwd_ws_bytes(int64_t R, int64_t d);
int layernorm_plan(int64_t R, int64_t d, int x_dt, int backward, int32_t out[4]);
int launch_layernorm_bwd(const void* G, int64_t g_ld, const void* X, int x_dt, int64_t x_ld, void* dX, int dx_dt,
                         int64_t dx_ld, int R, int d, const void* gamma, int gb_dt, const float* mean,
                         const float* rinv, float eps, int eps_inside, int stat, void* dgamma, void* dbeta, int dg_dt,
                         const float* g_scale, const float* x_scale, const float* gamma_scale, float* dx_scale,
                         float* dgamma_scale, float* dbeta_scale, const float* stat_in, int exact, void* ws,
                         cudaStream_t st);
size_t adam_ws_bytes(int64_t n_tensors);
// Every scale word the step WRITES (m, v, w, w_cast of every tensor) must be a different word, and none of them a
// gradient's scale word: the kernels read and write them concurrently.  `scratch` holds 4 * n_tensors pointers.
int check_adam_scale_words(int n_tensors, const scalify_array* grads, const scalify_array* m, const scalify_array* v,
                           const scalify_array* w, const scalify_array* w_cast, const void** scratch);
int launch_adam(int n_tensors, const scalify_array* grads, scalify_array* m, scalify_array* v, scalify_array* w,
                const scalify_array* w_cast,
                const int64_t* numel, float lr, float beta1, float beta2, float eps, int64_t step, void* ws,
                cudaStream_t st);

int launch_embedding_fwd(const long long* ids, long long n, int seq_len, int d, long long vocab, const void* wte,
                         const void* wpe, int w_dt, const float* wte_scale, const float* wpe_scale, void* Y, int y_dt,
                         float* y_scale, uint32_t* status, cudaStream_t st);
int launch_embedding_bwd(const long long* ids, long long n, int seq_len, int d, long long vocab, const void* dY, int g_dt,
                         const float* dy_scale, float* dwte, float* dwte_scale, float* dwpe, float* dwpe_scale,
                         cudaStream_t st);
int launch_softmax_fwd(const void* S, int s_dt, void* P, int p_dt, long long rows, int Tq, int Tk, int causal,
                       const float* s_scale, float* p_scale, cudaStream_t st);
int launch_softmax_bwd(const void* dP, int g_dt, const void* P, int p_dt, void* dS, int o_dt, long long rows, int Tk,
                       const float* dp_scale, const float* p_scale, float* ds_scale, cudaStream_t st);
size_t cross_entropy_ws_bytes(int64_t n);
size_t colsum_ws_bytes(int64_t N);
int launch_cast_colsum(const void* X, int x_dt, long long ld, long long R, long long N, const float* x_scale, void* C,
                       int c_dt, long long ldc, float* c_scale, void* Y, int y_dt, float* y_scale, void* ws,
                       cudaStream_t st);
int launch_colsum(const void* X, int x_dt, long long ld, long long R, long long N, const float* x_scale, void* Y, int y_dt,
                  float* y_scale, void* ws, cudaStream_t st);
int launch_cross_entropy(const void* logits, int l_dt, long long ld, int n_classes, const long long* targets, long long n,
                         const float* l_scale, float* loss, void* dlogits, int g_dt, float* g_scale, void* ws,
                         cudaStream_t st);

struct MatmulArgs {
  const void* A; int a_dt; int transA; int64_t lda, a_bs;
  const void* B; int b_dt; int transB; int64_t ldb, b_bs;
  void* Y; int y_dt; int64_t ldy, y_bs;
  int M, N, K, batch;
  const float* a_scale; const float* b_scale; float* y_scale;
  int stat;
  const float* stat_in;  // delayed rescale: earlier statistic (device) or NULL
  int force_ncta;  // 0: choose; 1: force the one-CTA kernel
  // speculative rescale: predicted statistic (device) or NULL; then Yq (FP8, dense like Y) is written by the GEMM
  const float* stat_hint;
  void* Yq; int q_dt;
  // stat_hint came from the library itself (the workspace header), not from the caller: a product that is better
  // split over K ignores it.  *took_spec (optional) reports whether the speculative kernel ran.
  int hint_optional;
  int* took_spec;
  // FP8-only form: Y is not stored (y_dt still names the 16-bit format the values are rounded through); the GEMM
  // publishes Yq's scale word and the next prediction itself, and a repair launch of the same kernel follows.
  int noy;
  float* yq_scale;
  float* hint_out;
  const void* bias; int bias_dt; const float* bias_scale;  // optional [N] vector added in the epilogue (add rule)
  float alpha_override;  // 0: the data component is divided by kf(K); otherwise multiplied by this (split-K partials)
  int no_split;          // 1: never split the contraction (the partial products of a split call)
};
size_t matmul_ws_bytes(int64_t rows, int64_t cols);
size_t matmul_splitk_ws_bytes(int64_t rows, int64_t cols);
int launch_bf16_round(const float* x, float* y, long long n, int two_wide, cudaStream_t st);
int host_state_selftest();
// debug build only (SCALIFY_ERR_UNSUPPORTED otherwise): violations seen since the last report
int debug_bounds_report(unsigned long long out[3], int reset_ranges, long long limit);
void map_cache_counters(unsigned long long* hits, unsigned long long* misses);
int launch_expire_wait(void* ws, unsigned long long limit_ns, uint32_t* waited_us, cudaStream_t st);
int launch_scaled_matmul(const MatmulArgs& a, void* ws, size_t ws_bytes, cudaStream_t st);
// Block-scaled matmul: A [M,K], B [N,K] FP8 row-major (dense), exponents in 128-row x 4-block tiles.
struct MxMatmulArgs {
  const void* A; int a_dt; const uint8_t* sfa;
  const void* B; int b_dt; const uint8_t* sfb;
  void* Y; int y_dt; int64_t ldy;
  int M, N, K;
  const float* a_scale; const float* b_scale; float* y_scale;
  int stat;
  int force_ncta;  // 0: choose; 1: force the one-CTA kernel
  int transA, transB;  // operand stored [K, rows]: consumed MN-major
};
int launch_mx_matmul(const MxMatmulArgs& a, void* ws, cudaStream_t st);
size_t mx_sf_bytes(int64_t rows, int64_t K);
struct AttentionArgs {
  const void* Q; const void* K; const void* V; int q_dt, k_dt, v_dt;   // FP8 [heads, T, hd] views
  int64_t q_ld, q_hs, k_ld, k_hs, v_ld, v_hs;                         // row and head strides in elements
  int64_t q_bs, k_bs, v_bs, o_bs;                                     // batch strides in elements
  void* O; int o_dt; int64_t o_ld, o_hs;                              // [heads, Tq, hd], F16 / BF16
  int batch, heads, Tq, Tk, hd;                                       // heads per batch element
  int causal;
  float sm_scale;
  const float* q_scale; const float* k_scale; const float* v_scale; float* o_scale;
  void* S_dump;  // optional BF16 [heads, Tq, Tk] dense: the scores' data component as rounded
  void* P_dump;  // optional E4M3 [heads, Tq, Tk] dense: the probabilities as fed to the second matmul
  uint32_t* status;
};
int launch_attention(const AttentionArgs& a, cudaStream_t st);

struct AttentionBwdArgs {
  const void* Q; const void* K; const void* V; const void* dO; int q_dt, k_dt, v_dt, do_dt;  // FP8 [heads, T, hd] views
  int64_t q_ld, q_hs, k_ld, k_hs, v_ld, v_hs, do_ld, do_hs;                                  // strides in elements
  int64_t q_bs, k_bs, v_bs, do_bs, dq_bs, dk_bs, dv_bs;                                      // batch strides
  const void* P;   // E4M3 [heads, Tq, Tk] dense: the probabilities the forward pass used
  void* dS;        // E5M2 [heads, Tq, Tk] dense (output, and operand of the dK product)
  void* dQ; void* dK; void* dV; int g_dt;   // F16 / BF16 / F32 [heads, T, hd] views
  int64_t dq_ld, dq_hs, dk_ld, dk_hs, dv_ld, dv_hs;
  int batch, heads, Tq, Tk, hd;   // heads per batch element
  int causal;
  float sm_scale;  // a power of two
  const float* q_scale; const float* k_scale; const float* v_scale; const float* p_scale; const float* do_scale;
  float* ds_scale; float* dq_scale; float* dk_scale; float* dv_scale;
  void* dP_dump;   // optional BF16 [heads, Tq, Tk] dense: dP's data component as rounded
  uint32_t* status;
};
int launch_attention_bwd(const AttentionBwdArgs& a, cudaStream_t st);
int launch_mx_quantize_t(const void* X, int x_dt, int64_t rows, int64_t K, int64_t ldx, void* data, int elem_dt,
                         uint8_t* sf, const float* x_scale, float* y_scale, uint32_t* status, cudaStream_t st);
int launch_mx_quantize(const void* X, int x_dt, int64_t rows, int64_t K, int64_t ldx, void* data, int elem_dt,
                       uint8_t* sf, const float* x_scale, float* y_scale, uint32_t* status, cudaStream_t st);

}  // namespace scalify
