// Shared declarations of the CUDA library: policy handle, per-layer device records,
// launch helpers.  Nothing here is visible through the C ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/actorq.h"

#define ACTORQ_MAX_LAYERS 16
#define ACTORQ_MAX_K 16384

namespace actorq {

// Per-layer numbers that only exist after the device has reduced the weight range.
// Written by round_kernel (from the reduced weight range), read by every forward kernel.
struct LayerParams {
  float s_w;      // weight delta (Eq. 2)
  int z_w;        // weight zero-point
  float s_a;      // input activation delta
  int z_a;        // input activation zero-point
  float inv_s_a;  // 1 / s_a, the multiplier of the input quantizer
  float P;        // s_a * s_w : real value of one accumulator unit
  float M;        // P / s_out : hidden-layer requantization multiplier
  int z_out;      // zero-point of the next layer's input (ReLU floor)
  int bias_absmax; // max_n |bias_q[n]| (bounds the accumulator magnitude)
};

struct LayerGeom {
  int kind;                                   // actorq_layer_kind
  int K;                                      // reduction length: in_features or in_c*kh*kw
  int N;                                      // output features (FC) or output channels (conv)
  int in_c, in_h, in_w, out_c, kh, kw, stride, out_h, out_w;
  long long in_elems, out_elems;              // per observation
  long long w_elems;                          // N * K
  int per_channel;                            // 1: every output channel has its own weight delta / zero-point
};

struct ActParams { float s; int z; float inv_s; };

struct LayerDev {
  LayerGeom g;
  const float *w_f32;   // caller's fp32 weights (valid during quantize only)
  const float *b_f32;
  int8_t *wq;           // int8 codes in the caller's element order, [N][K]
  int8_t *wq_img;       // tensor-core image: K-major 128-byte-swizzled tiles (see mlp_fused.cu)
  int *colsum;          // [N] sum_k wq[n][k]
  int *bias_q;          // [N]
  int *colconst;        // [N] bias_q - z_a*colsum + K*z_a*z_w
  // per-output-channel quantization (per_channel layers): channel n's weight delta and zero-point,
  // accumulator unit P[n] = s_a * s_w[n] and requantization multiplier M[n] = P[n] / s_out
  float *ch_sw;         // [N]
  int *ch_zw;           // [N]
  float *ch_P;          // [N]
  float *ch_M;          // [N]
  int *koff;            // conv-GEMM path: receptive-field offset of each 16 (4) bytes of K
  int perm_c, perm_kh, perm_kw;   // weight-image K order (kh, kw, c) instead of (c, kh, kw); 0 = caller's order
  long long img_bytes;
};

}  // namespace actorq

struct actorq_policy {
  int n_layers;
  int head;
  int obs_dtype;
  int device;
  actorq::LayerDev layers[ACTORQ_MAX_LAYERS];
  actorq::ActParams act[ACTORQ_MAX_LAYERS + 1];   // activation quantizers (host copy)
  actorq::LayerParams *d_params;                  // [n_layers] device
  int *d_rangekeys;                               // [2 sets][ACTORQ_MAX_LAYERS][2] ordered-int range accumulators
  int range_parity;                               // which set the next quantize call reduces into
  int *d_status;                                  // device status word (sticky until read)
  void *pool;                                     // one allocation holding all of the above
  // scratch for architectures whose activations live in device memory
  int8_t *scratch[2];
  long long scratch_elems;
  // activation operand blocks and row-sum counters of the layer-at-a-time CTA-pair path (fc_pair.cu)
  void *fcp_mem;
  long long fcp_rows;
  int fcp_ok;                                     // 1 if that path takes the policy (its layers then have weight images)
  int launches;
  int fused_ok;                                   // 1 if the fused tcgen05 MLP kernel applies
  int fused_variant;                              // 0: pick (resident-weights kernel for small policies, else CTA pairs when
                                                  // possible), 1: single-CTA kernel, 2: CTA pairs with the weight ring,
                                                  // 3: one launch per layer on CTA pairs (fc_pair.cu), 4: resident-weights kernel
  int conv_ok;                                    // 1 if the tcgen05 implicit-GEMM layer kernel applies
  int sm_count;
  // staging of actorq_policy_forward_host: kHostSlots chunks in flight (device copies of a chunk's
  // observations / outputs / actions), two copy streams, events that order the three stages
  static const int kHostSlots = 3;
  void *hs_mem;                                   // one allocation holding every slot
  void *hs_obs[kHostSlots];
  float *hs_out[kHostSlots];
  int *hs_act[kHostSlots];
  long long hs_rows;                              // rows per slot
  cudaStream_t hs_in, hs_outs;                    // host -> device, device -> host
  cudaEvent_t hs_ev_in[kHostSlots], hs_ev_comp[kHostSlots], hs_ev_out[kHostSlots];
  int hs_ready;
  // set by actorq_policy_forward_explore around its forward: per-row sigma [batch] and standard normal
  // draws [batch][out_dim]; a forward kernel that applies them in its head sets ex_applied
  const float *ex_sigma, *ex_noise;
  int ex_applied;
  // actorq_policy_forward_explore_seeded: the draws come from the counter-based generator of
  // explore_rng.cuh instead (ex_noise is then nullptr), keyed by ex_seed and the absolute row ex_row0 + b
  int ex_seeded;
  unsigned long long ex_seed;
  long long ex_row0;
  // the fp16 actor (fp16_pair.cu): precision 16 = the policy was cast to binary16 (actorq_cast_params_fp16),
  // otherwise quantized to int8.  Its own pool (status block, binary16 weight images, binary32 biases) and
  // two activation buffers grown on demand.
  int precision;
  void *f16_pool;
  uint8_t *f16_img[ACTORQ_MAX_LAYERS];
  float *f16_bias[ACTORQ_MAX_LAYERS];
  void *f16_act;
  long long f16_rows;
};

namespace actorq {

int launch_quantize(actorq_policy *p, cudaStream_t st);
long long blob_bytes(const actorq_policy *p);
int launch_export_blob(actorq_policy *p, void *blob, cudaStream_t st);
int launch_import_blob(actorq_policy *p, const void *blob, cudaStream_t st);
int launch_forward_generic(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                           int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st);
// fused tcgen05 path (mlp_fused.cu)
bool fused_mlp_supported(const actorq_policy *p);
long long fused_image_bytes(const LayerGeom &g);
int launch_forward_fused(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                         int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st);

// the same on CTA pairs, tcgen05 cta_group::2 (mlp_fused_pair.cu)
bool fused_pair_supported(const actorq_policy *p);
int launch_forward_fused_pair(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                              int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st);

// small policies with all weights resident in shared memory, two tiles in flight per CTA pair (mlp_resident.cu)
bool fused_resident_supported(const actorq_policy *p);
int launch_forward_fused_resident(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                                  int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st);

// wide all-FC policies, one launch per layer on CTA pairs (fc_pair.cu)
bool fc_pair_supported(const actorq_policy *p);
int launch_forward_fc_pair(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                           int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st);

// the fully connected tail of a convolutional policy on the layer kernel of fc_pair.cu
int fc_tail_begin(actorq_policy *p, int l_begin, long long batch, cudaStream_t st, int8_t **blocks, int *nkb, int **rowsums,
                  int clear_here, int **rs_all, long long *rs_all_len);
// convolution layers with their input staged in shared memory (conv_staged.cu)
bool conv_staged_supported(const actorq_policy *p, int l, long long batch);
int launch_conv_staged(actorq_policy *p, int l, const void *in, long long batch, int8_t *out_act,
                       int8_t *blk_out, int *blk_rs, int blk_nkb, int blk_unsigned, int *zero_ptr, long long zero_len,
                       int *dbg_acc, int8_t *dbg_act, cudaStream_t st);
int fc_tail_run(actorq_policy *p, int l_begin, long long batch, float *out, int *actions,
                int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st);

// the fp16 actor (fp16_pair.cu)
bool fp16_supported(const actorq_policy *p);
int fp16_setup(actorq_policy *p);
int launch_cast_fp16(actorq_policy *p, cudaStream_t st);
int launch_forward_fp16(actorq_policy *p, const void *obs, long long batch, float *out, int *actions, cudaStream_t st);

// out[b][n] = clamp(out[b][n] + sigma[b] * noise[b][n], -1, 1) for the paths whose head does not do it
int launch_explore(float *out, const float *sigma, const float *noise, long long batch, int out_dim, int sm_count, cudaStream_t st);
int launch_explore_seeded(float *out, const float *sigma, unsigned long long seed, long long row0, long long batch, int out_dim,
                          int sm_count, cudaStream_t st);
int launch_selftest_bounded_wait(actorq_policy *p, long long limit_ns, cudaStream_t st);
int launch_selftest_int8_mma_peak(actorq_policy *p, long long groups, int a_in_tmem, long long *ops, cudaStream_t st);
// tcgen05 implicit-GEMM conv / FC layers (conv_gemm.cu)
bool conv_gemm_supported(const actorq_policy *p);
bool conv_gemm_image_perm(const actorq_policy *p, int l, int *C, int *KH, int *KW);
int conv_gemm_koff_entries(const actorq_policy *p, int l);
void conv_gemm_fill_koff(const actorq_policy *p, int l, int *koff);
int launch_forward_conv_gemm(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                             int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st);

static inline int cuda_ok(cudaError_t e) { return e == cudaSuccess ? ACTORQ_OK : ACTORQ_ERR_CUDA; }

}  // namespace actorq
