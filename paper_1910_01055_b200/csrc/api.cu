// C ABI of the library (declared in include/actorq.h): argument checking, the policy handle and
// its single device allocation, and dispatch to the quantizer and forward kernels.
#include <math.h>
#include <new>
#include <string.h>
#include "common.cuh"

using namespace actorq;

namespace {

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// activation quantizer of one layer input from its calibration range: the weight rule (Eq. 2)
// applied to (min, max); binary32 throughout, round half to even
ActParams act_from_range(float rmin, float rmax) {
  ActParams a;
  float lo = fminf(rmin, 0.0f), hi = fmaxf(rmax, 0.0f);
  volatile float span = hi - lo;
  volatile float s = span / 255.0f;
  if (!(s > 0.0f)) { a.s = 1.0f; a.z = 0; a.inv_s = 1.0f; return a; }
  volatile float zf = (-lo) / s;
  long z = lrintf(zf) - 128;
  a.s = s;
  a.z = (int)(z < -128 ? -128 : (z > 127 ? 127 : z));
  volatile float inv = 1.0f / s;
  a.inv_s = inv;
  return a;
}

int fill_geometry(const actorq_layer_desc &d, LayerGeom &g) {
  memset(&g, 0, sizeof(g));
  g.kind = d.kind;
  if (d.kind == ACTORQ_FC) {
    if (d.in_features <= 0 || d.out_features <= 0) return ACTORQ_ERR_INVALID_ARG;
    g.K = d.in_features;
    g.N = d.out_features;
    g.in_elems = g.K;
    g.out_elems = g.N;
  } else if (d.kind == ACTORQ_CONV2D) {
    if (d.in_c <= 0 || d.in_h <= 0 || d.in_w <= 0 || d.out_c <= 0 || d.kh <= 0 || d.kw <= 0 || d.stride <= 0)
      return ACTORQ_ERR_INVALID_ARG;
    if (d.kh > d.in_h || d.kw > d.in_w) return ACTORQ_ERR_INVALID_ARG;
    g.in_c = d.in_c; g.in_h = d.in_h; g.in_w = d.in_w;
    g.out_c = d.out_c; g.kh = d.kh; g.kw = d.kw; g.stride = d.stride;
    g.out_h = (d.in_h - d.kh) / d.stride + 1;
    g.out_w = (d.in_w - d.kw) / d.stride + 1;
    g.K = d.in_c * d.kh * d.kw;
    g.N = d.out_c;
    g.in_elems = (long long)d.in_c * d.in_h * d.in_w;
    g.out_elems = (long long)d.out_c * g.out_h * g.out_w;
  } else {
    return ACTORQ_ERR_INVALID_ARG;
  }
  if (g.K > ACTORQ_MAX_K) return ACTORQ_ERR_UNSUPPORTED;
  g.w_elems = (long long)g.N * g.K;
  if (d.per_channel != 0 && d.per_channel != 1) return ACTORQ_ERR_INVALID_ARG;
  g.per_channel = d.per_channel;
  return ACTORQ_OK;
}

bool same_geometry(const LayerGeom &a, const LayerGeom &b) { return memcmp(&a, &b, sizeof(LayerGeom)) == 0; }

int ensure_scratch(actorq_policy *p, long long batch) {
  long long per_row = 0;
  for (int l = 0; l < p->n_layers; ++l) {
    if (p->layers[l].g.in_elems > per_row) per_row = p->layers[l].g.in_elems;
    if (p->layers[l].g.out_elems > per_row) per_row = p->layers[l].g.out_elems;
  }
  per_row = (per_row + 15) / 16 * 16;            // rows of the all-FC tensor-core path are 16-byte aligned
  long long need = batch * per_row;
  if (need <= p->scratch_elems) return ACTORQ_OK;
  if (p->scratch[0]) cudaFree(p->scratch[0]);
  p->scratch[0] = p->scratch[1] = nullptr;
  p->scratch_elems = 0;
  size_t one = align_up((size_t)need, 256);
  void *mem = nullptr;
  if (cudaMalloc(&mem, 2 * one) != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_NOMEM; }
  p->scratch[0] = (int8_t *)mem;
  p->scratch[1] = (int8_t *)mem + one;
  p->scratch_elems = need;
  return ACTORQ_OK;
}

int create_policy(const actorq_layer_desc *layers, int n_layers, int head, int obs_dtype, actorq_policy **out) {
  actorq_policy *p = new (std::nothrow) actorq_policy;
  if (!p) return ACTORQ_ERR_NOMEM;
  memset(p, 0, sizeof(*p));
  p->n_layers = n_layers;
  p->head = head;
  p->obs_dtype = obs_dtype;
  if (cudaGetDevice(&p->device) != cudaSuccess) { delete p; return ACTORQ_ERR_CUDA; }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, p->device) != cudaSuccess) { delete p; return ACTORQ_ERR_CUDA; }
  p->sm_count = prop.multiProcessorCount;
  for (int l = 0; l < n_layers; ++l) {
    int rc = fill_geometry(layers[l], p->layers[l].g);
    if (rc != ACTORQ_OK) { delete p; return rc; }
    if (l > 0 && p->layers[l].g.in_elems != p->layers[l - 1].g.out_elems) { delete p; return ACTORQ_ERR_INVALID_ARG; }
  }
  p->fused_ok = fused_mlp_supported(p) ? 1 : 0;
  p->conv_ok = (!p->fused_ok && conv_gemm_supported(p)) ? 1 : 0;
  // per-channel layers: the fused MLP epilogues take one multiplier and one weight zero-point per
  // layer, so such policies use the conv-GEMM layer kernel (which reads them per column) where it
  // applies, else the layer-at-a-time kernels
  for (int l = 0; l < n_layers; ++l)
    if (p->layers[l].g.per_channel) p->fused_ok = 0;
  if (p->fused_ok == 0 && p->conv_ok == 0) p->conv_ok = conv_gemm_supported(p) ? 1 : 0;
  p->fcp_ok = fc_pair_supported(p) ? 1 : 0;

  // one pool: params, range keys, status, then per layer codes / image / per-output ints
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
  size_t o_params = take(sizeof(LayerParams) * n_layers);
  size_t o_keys = take(sizeof(int) * 4 * ACTORQ_MAX_LAYERS);
  size_t o_status = take(sizeof(int) * 16);     // status word + where a timed-out wait gave up
  size_t o_wq[ACTORQ_MAX_LAYERS], o_img[ACTORQ_MAX_LAYERS], o_ints[ACTORQ_MAX_LAYERS], o_koff[ACTORQ_MAX_LAYERS];
  for (int l = 0; l < n_layers; ++l) {
    LayerDev &L = p->layers[l];
    o_wq[l] = take((size_t)L.g.w_elems);
    L.img_bytes = (p->fused_ok || p->conv_ok || p->fcp_ok) ? fused_image_bytes(L.g) : 0;
    o_img[l] = take((size_t)L.img_bytes);
    o_ints[l] = take(sizeof(int) * 7 * align_up((size_t)L.g.N, 128));   // zero-padded to 128 entries
    o_koff[l] = take(p->conv_ok ? sizeof(int) * (size_t)conv_gemm_koff_entries(p, l) : 0);
  }
  if (cudaMalloc(&p->pool, off) != cudaSuccess) { cudaGetLastError(); delete p; return ACTORQ_ERR_NOMEM; }
  if (cudaMemset(p->pool, 0, off) != cudaSuccess) { cudaFree(p->pool); delete p; return ACTORQ_ERR_CUDA; }
  char *base = (char *)p->pool;
  p->d_params = (LayerParams *)(base + o_params);
  p->d_rangekeys = (int *)(base + o_keys);
  p->d_status = (int *)(base + o_status);
  for (int l = 0; l < n_layers; ++l) {
    LayerDev &L = p->layers[l];
    L.wq = (int8_t *)(base + o_wq[l]);
    L.wq_img = L.img_bytes ? (int8_t *)(base + o_img[l]) : nullptr;
    L.colsum = (int *)(base + o_ints[l]);
    L.bias_q = L.colsum + align_up((size_t)L.g.N, 128);
    L.colconst = L.bias_q + align_up((size_t)L.g.N, 128);
    L.ch_sw = (float *)(L.colconst + align_up((size_t)L.g.N, 128));
    L.ch_zw = (int *)(L.ch_sw + align_up((size_t)L.g.N, 128));
    L.ch_P = (float *)(L.ch_zw + align_up((size_t)L.g.N, 128));
    L.ch_M = L.ch_P + align_up((size_t)L.g.N, 128);
    L.koff = nullptr;
    L.perm_c = L.perm_kh = L.perm_kw = 0;
    if (p->conv_ok) {
      L.koff = (int *)(base + o_koff[l]);
      const int n_ent = conv_gemm_koff_entries(p, l);
      int *tmp = new (std::nothrow) int[n_ent];
      if (!tmp) { cudaFree(p->pool); delete p; return ACTORQ_ERR_NOMEM; }
      conv_gemm_fill_koff(p, l, tmp);
      cudaError_t e = cudaMemcpy(L.koff, tmp, sizeof(int) * n_ent, cudaMemcpyHostToDevice);
      delete[] tmp;
      if (e != cudaSuccess) { cudaFree(p->pool); delete p; return ACTORQ_ERR_CUDA; }
      int C, KH, KW;
      if (conv_gemm_image_perm(p, l, &C, &KH, &KW)) { L.perm_c = C; L.perm_kh = KH; L.perm_kw = KW; }
    }
  }
  *out = p;
  return ACTORQ_OK;
}

}  // namespace

extern "C" {

int actorq_quantize_params(const actorq_layer_desc *layers, int n_layers, const actorq_range *input_ranges,
                           int head, int obs_dtype, void *cuda_stream, actorq_policy **inout_policy) {
  if (!layers || !input_ranges || !inout_policy) return ACTORQ_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > ACTORQ_MAX_LAYERS) return ACTORQ_ERR_INVALID_ARG;
  if (head < ACTORQ_HEAD_TANH || head > ACTORQ_HEAD_LINEAR) return ACTORQ_ERR_INVALID_ARG;
  if (obs_dtype != ACTORQ_OBS_F32 && obs_dtype != ACTORQ_OBS_U8_DIV255) return ACTORQ_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    if (!layers[l].weight) return ACTORQ_ERR_INVALID_ARG;
    if (!(input_ranges[l].min <= input_ranges[l].max)) {          // also rejects NaN
      if (!(l == 0 && obs_dtype == ACTORQ_OBS_U8_DIV255)) return ACTORQ_ERR_INVALID_ARG;
    }
    if (isinf(input_ranges[l].min) || isinf(input_ranges[l].max)) return ACTORQ_ERR_INVALID_ARG;
  }
  actorq_policy *p = *inout_policy;
  if (p != nullptr && p->precision == 16) return ACTORQ_ERR_INVALID_ARG;      // a policy cast to binary16 is re-cast, not quantized
  if (p == nullptr) {
    int rc = create_policy(layers, n_layers, head, obs_dtype, &p);
    if (rc != ACTORQ_OK) return rc;
  } else {
    if (p->n_layers != n_layers || p->head != head || p->obs_dtype != obs_dtype) return ACTORQ_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l) {
      LayerGeom g;
      int rc = fill_geometry(layers[l], g);
      if (rc != ACTORQ_OK) return rc;
      if (!same_geometry(g, p->layers[l].g)) return ACTORQ_ERR_INVALID_ARG;
    }
  }
  for (int l = 0; l < n_layers; ++l) {
    p->layers[l].w_f32 = layers[l].weight;
    p->layers[l].b_f32 = layers[l].bias;
    if (l == 0 && obs_dtype == ACTORQ_OBS_U8_DIV255) {
      volatile float s = 1.0f / 255.0f;
      p->act[0].s = s; p->act[0].z = -128; p->act[0].inv_s = 255.0f;
    } else {
      p->act[l] = act_from_range(input_ranges[l].min, input_ranges[l].max);
    }
  }
  p->act[n_layers].s = 1.0f; p->act[n_layers].z = 0; p->act[n_layers].inv_s = 1.0f;
  int rc = launch_quantize(p, (cudaStream_t)cuda_stream);
  for (int l = 0; l < n_layers; ++l) { p->layers[l].w_f32 = nullptr; p->layers[l].b_f32 = nullptr; }
  if (rc != ACTORQ_OK) {
    if (*inout_policy == nullptr) actorq_free(p);
    return rc;
  }
  *inout_policy = p;
  return ACTORQ_OK;
}

static int forward_impl(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                        int dbg_layer, int *dbg_acc, signed char *dbg_act, void *cuda_stream) {
  if (!p) return ACTORQ_ERR_INVALID_ARG;
  if (batch < 0) return ACTORQ_ERR_INVALID_ARG;
  p->launches = 0;
  if (batch == 0) return ACTORQ_OK;
  if (!obs || !out) return ACTORQ_ERR_INVALID_ARG;
  if (p->head == ACTORQ_HEAD_ARGMAX && !actions) return ACTORQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(obs) & 15) != 0) return ACTORQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (p->precision == 16) {             // a policy cast to binary16: its own layer kernel, no debug taps
    if (dbg_layer >= 0) return ACTORQ_ERR_UNSUPPORTED;
    return launch_forward_fp16(p, obs, batch, out, actions, st);
  }
  // Wide all-FC policies (and any all-FC policy when the caller asks for it): one launch per layer
  // on CTA pairs, activations as MMA operand blocks in device memory.  With a hidden layer wider than
  // 512 the fused kernels hold one accumulator per tile (their tensor memory also carries the
  // activations) and pause the MMAs at every hand-over; the layer kernel alternates two accumulators
  // and spreads a layer's (row tile, column chunk) items over all CTA pairs, which wins from a few
  // thousand rows up to the largest batches.
  bool wide = false;
  for (int l = 0; l + 1 < p->n_layers; ++l) wide = wide || p->layers[l].g.N > 512;
  if ((p->fused_variant == 3 || !p->fused_ok || (p->fused_variant == 0 && wide)) && p->fcp_ok) {
    const int rc = launch_forward_fc_pair(p, obs, batch, out, actions, dbg_layer, dbg_acc, (int8_t *)dbg_act, st);
    if (rc != ACTORQ_ERR_UNSUPPORTED || p->fused_variant == 3) return rc;
    p->launches = 0;
  }
  if (p->fused_ok) {
    // small policies: the whole int8 policy resident in shared memory, two tiles in flight
    if ((p->fused_variant == 0 || p->fused_variant == 4) && fused_resident_supported(p)) {
      const int rc = launch_forward_fused_resident(p, obs, batch, out, actions, dbg_layer, dbg_acc, (int8_t *)dbg_act, st);
      if (rc != ACTORQ_ERR_UNSUPPORTED || p->fused_variant == 4) return rc;
      p->launches = 0;
    }
    // CTA pairs (n = 256 MMAs, half the weight traffic per SM) unless the caller pinned the
    // single-CTA kernel or the device cannot co-schedule pairs
    if (p->fused_variant != 1 && fused_pair_supported(p)) {
      const int rc = launch_forward_fused_pair(p, obs, batch, out, actions, dbg_layer, dbg_acc, (int8_t *)dbg_act, st);
      if (rc != ACTORQ_ERR_UNSUPPORTED || p->fused_variant == 2) return rc;
      p->launches = 0;
    }
    return launch_forward_fused(p, obs, batch, out, actions, dbg_layer, dbg_acc, (int8_t *)dbg_act, st);
  }
  int rc = ensure_scratch(p, batch);
  if (rc != ACTORQ_OK) return rc;
  if (p->conv_ok)
    return launch_forward_conv_gemm(p, obs, batch, out, actions, dbg_layer, dbg_acc, (int8_t *)dbg_act, st);
  return launch_forward_generic(p, obs, batch, out, actions, dbg_layer, dbg_acc, (int8_t *)dbg_act, st);
}

int actorq_cast_params_fp16(const actorq_layer_desc *layers, int n_layers, int head, int obs_dtype, void *cuda_stream,
                            actorq_policy **inout_policy) {
  if (!layers || !inout_policy) return ACTORQ_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > ACTORQ_MAX_LAYERS) return ACTORQ_ERR_INVALID_ARG;
  if (head < ACTORQ_HEAD_TANH || head > ACTORQ_HEAD_LINEAR) return ACTORQ_ERR_INVALID_ARG;
  if (obs_dtype != ACTORQ_OBS_F32 && obs_dtype != ACTORQ_OBS_U8_DIV255) return ACTORQ_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!layers[l].weight) return ACTORQ_ERR_INVALID_ARG;
  actorq_policy *p = *inout_policy;
  if (p == nullptr) {
    p = new (std::nothrow) actorq_policy;
    if (!p) return ACTORQ_ERR_NOMEM;
    memset(p, 0, sizeof(*p));
    p->n_layers = n_layers; p->head = head; p->obs_dtype = obs_dtype; p->precision = 16;
    cudaDeviceProp prop;
    if (cudaGetDevice(&p->device) != cudaSuccess || cudaGetDeviceProperties(&prop, p->device) != cudaSuccess) { delete p; return ACTORQ_ERR_CUDA; }
    p->sm_count = prop.multiProcessorCount;
    for (int l = 0; l < n_layers; ++l) {
      int rc = fill_geometry(layers[l], p->layers[l].g);
      if (rc == ACTORQ_OK && l > 0 && p->layers[l].g.in_elems != p->layers[l - 1].g.out_elems) rc = ACTORQ_ERR_INVALID_ARG;
      if (rc != ACTORQ_OK) { delete p; return rc; }
    }
    if (!fp16_supported(p)) { delete p; return ACTORQ_ERR_UNSUPPORTED; }
    const int rc = fp16_setup(p);
    if (rc != ACTORQ_OK) { actorq_free(p); return rc; }
  } else {
    if (p->precision != 16 || p->n_layers != n_layers || p->head != head || p->obs_dtype != obs_dtype) return ACTORQ_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l) {
      LayerGeom g;
      const int rc = fill_geometry(layers[l], g);
      if (rc != ACTORQ_OK) return rc;
      if (!same_geometry(g, p->layers[l].g)) return ACTORQ_ERR_INVALID_ARG;
    }
  }
  for (int l = 0; l < n_layers; ++l) { p->layers[l].w_f32 = layers[l].weight; p->layers[l].b_f32 = layers[l].bias; }
  const int rc = launch_cast_fp16(p, (cudaStream_t)cuda_stream);
  for (int l = 0; l < n_layers; ++l) { p->layers[l].w_f32 = nullptr; p->layers[l].b_f32 = nullptr; }
  if (rc != ACTORQ_OK) {
    if (*inout_policy == nullptr) actorq_free(p);
    return rc;
  }
  *inout_policy = p;
  return ACTORQ_OK;
}

int actorq_policy_forward(actorq_policy *policy, const void *obs, long long batch, float *out, int *actions,
                          void *cuda_stream) {
  return forward_impl(policy, obs, batch, out, actions, -1, nullptr, nullptr, cuda_stream);
}

int actorq_policy_forward_explore(actorq_policy *p, const void *obs, long long batch, const float *sigma, const float *noise,
                                  float *out, void *cuda_stream) {
  if (!p || batch < 0) return ACTORQ_ERR_INVALID_ARG;
  if (p->head != ACTORQ_HEAD_TANH) return ACTORQ_ERR_UNSUPPORTED;
  if (batch > 0 && (!sigma || !noise)) return ACTORQ_ERR_INVALID_ARG;
  p->ex_sigma = sigma; p->ex_noise = noise; p->ex_applied = 0;
  int rc = forward_impl(p, obs, batch, out, nullptr, -1, nullptr, nullptr, cuda_stream);
  const int applied = p->ex_applied;
  p->ex_sigma = p->ex_noise = nullptr; p->ex_applied = 0;
  if (rc != ACTORQ_OK || batch == 0 || applied) return rc;
  rc = actorq::launch_explore(out, sigma, noise, batch, (int)p->layers[p->n_layers - 1].g.out_elems, p->sm_count, (cudaStream_t)cuda_stream);
  p->launches++;
  return rc;
}

int actorq_policy_forward_explore_seeded(actorq_policy *p, const void *obs, long long batch, const float *sigma,
                                         unsigned long long seed, long long first_row, float *out, void *cuda_stream) {
  if (!p || batch < 0 || first_row < 0) return ACTORQ_ERR_INVALID_ARG;
  if (p->head != ACTORQ_HEAD_TANH) return ACTORQ_ERR_UNSUPPORTED;
  if (batch > 0 && !sigma) return ACTORQ_ERR_INVALID_ARG;
  p->ex_sigma = sigma; p->ex_noise = nullptr; p->ex_applied = 0;
  p->ex_seeded = 1; p->ex_seed = seed; p->ex_row0 = first_row;
  int rc = forward_impl(p, obs, batch, out, nullptr, -1, nullptr, nullptr, cuda_stream);
  const int applied = p->ex_applied;
  p->ex_sigma = nullptr; p->ex_applied = 0; p->ex_seeded = 0;
  if (rc != ACTORQ_OK || batch == 0 || applied) return rc;
  rc = actorq::launch_explore_seeded(out, sigma, seed, first_row, batch, (int)p->layers[p->n_layers - 1].g.out_elems, p->sm_count,
                                     (cudaStream_t)cuda_stream);
  p->launches++;
  return rc;
}

int actorq_policy_forward_debug(actorq_policy *policy, const void *obs, long long batch, float *out, int *actions,
                                int layer, int *acc, signed char *act_q, void *cuda_stream) {
  if (!policy || layer < 0 || layer >= policy->n_layers || !acc) return ACTORQ_ERR_INVALID_ARG;
  if (layer + 1 < policy->n_layers && !act_q) return ACTORQ_ERR_INVALID_ARG;
  return forward_impl(policy, obs, batch, out, actions, layer, acc, act_q, cuda_stream);
}

// Host-buffer forward: the batch is cut into chunks and three stages run on three streams, ordered
// by events: copy a chunk's observations in, run the forward on the caller's stream, copy its
// outputs back.  With pinned host memory the copies of neighbouring chunks overlap the compute.
static long long host_chunk_rows(const actorq_policy *p, long long batch) {
  const long long row_bytes = p->layers[0].g.in_elems * (p->obs_dtype == ACTORQ_OBS_F32 ? 4 : 1);
  long long rows = (8ll << 20) / (row_bytes > 0 ? row_bytes : 1);      // about 8 MB of observations per chunk
  rows = rows / 256 * 256;                                             // whole tile pairs
  if (rows < 256) rows = 256;
  return rows < batch ? rows : batch;
}

static int ensure_host_staging(actorq_policy *p, long long rows) {
  if (!p->hs_ready) {
    // all or nothing: whatever was created before a failure is destroyed again (the next call starts over)
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev[3 * actorq_policy::kHostSlots];
    int n_ev = 0;
    bool ok = cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) == cudaSuccess;
    for (; ok && n_ev < 3 * actorq_policy::kHostSlots; ++n_ev)
      if (cudaEventCreateWithFlags(&ev[n_ev], cudaEventDisableTiming) != cudaSuccess) { ok = false; break; }
    if (!ok) {
      for (int i = 0; i < n_ev; ++i) cudaEventDestroy(ev[i]);
      if (s_out) cudaStreamDestroy(s_out);
      if (s_in) cudaStreamDestroy(s_in);
      cudaGetLastError();
      return ACTORQ_ERR_CUDA;
    }
    p->hs_in = s_in; p->hs_outs = s_out;
    for (int i = 0; i < actorq_policy::kHostSlots; ++i) {
      p->hs_ev_in[i] = ev[3 * i]; p->hs_ev_comp[i] = ev[3 * i + 1]; p->hs_ev_out[i] = ev[3 * i + 2];
    }
    p->hs_ready = 1;
  }
  if (rows <= p->hs_rows) return ACTORQ_OK;
  if (p->hs_mem) { cudaDeviceSynchronize(); cudaFree(p->hs_mem); p->hs_mem = nullptr; p->hs_rows = 0; }
  const size_t obs_b = align_up((size_t)rows * (size_t)p->layers[0].g.in_elems * (p->obs_dtype == ACTORQ_OBS_F32 ? 4 : 1), 256);
  const size_t out_b = align_up((size_t)rows * (size_t)p->layers[p->n_layers - 1].g.out_elems * sizeof(float), 256);
  const size_t act_b = align_up((size_t)rows * sizeof(int), 256);
  void *mem = nullptr;
  if (cudaMalloc(&mem, actorq_policy::kHostSlots * (obs_b + out_b + act_b)) != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_NOMEM; }
  p->hs_mem = mem;
  char *c = (char *)mem;
  for (int i = 0; i < actorq_policy::kHostSlots; ++i) {
    p->hs_obs[i] = c; c += obs_b;
    p->hs_out[i] = (float *)c; c += out_b;
    p->hs_act[i] = (int *)c; c += act_b;
  }
  p->hs_rows = rows;
  return ACTORQ_OK;
}

int actorq_policy_forward_host(actorq_policy *p, const void *obs_host, long long batch, float *out_host, int *actions_host,
                               void *cuda_stream) {
  if (!p || batch < 0) return ACTORQ_ERR_INVALID_ARG;
  p->launches = 0;
  if (batch == 0) return ACTORQ_OK;
  if (!obs_host || !out_host) return ACTORQ_ERR_INVALID_ARG;
  const bool want_actions = p->head == ACTORQ_HEAD_ARGMAX;
  if (want_actions && !actions_host) return ACTORQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const long long rows = host_chunk_rows(p, batch);
  int rc = ensure_host_staging(p, rows);
  if (rc != ACTORQ_OK) return rc;
  const size_t obs_row = (size_t)p->layers[0].g.in_elems * (p->obs_dtype == ACTORQ_OBS_F32 ? 4 : 1);
  const size_t out_row = (size_t)p->layers[p->n_layers - 1].g.out_elems * sizeof(float);
  const int S = actorq_policy::kHostSlots;
  // The forwards run on the caller's stream, behind everything enqueued on it before this call (a
  // re-quantize, say).  The copies in wait only for their staging slot: the host observations are
  // ready when the call is made, so the first copies of this call overlap the tail of the previous one.
  int launches = 0;
  long long done = 0;
  int n_chunks = 0;
  for (long long r0 = 0; r0 < batch; r0 += rows, ++n_chunks) {
    const int slot = n_chunks % S;
    const long long n = (batch - r0 < rows) ? batch - r0 : rows;
    // the slot's observations were last read by the forward of the chunk that used it before, its
    // outputs by that chunk's copy-out
    // (events of earlier calls count too; waiting on an event that was never recorded is a no-op)
    if (cudaStreamWaitEvent(p->hs_in, p->hs_ev_comp[slot], 0) != cudaSuccess) return ACTORQ_ERR_CUDA;
    if (cudaStreamWaitEvent(st, p->hs_ev_out[slot], 0) != cudaSuccess) return ACTORQ_ERR_CUDA;
    if (cudaMemcpyAsync(p->hs_obs[slot], (const char *)obs_host + (size_t)r0 * obs_row, (size_t)n * obs_row,
                        cudaMemcpyHostToDevice, p->hs_in) != cudaSuccess) return ACTORQ_ERR_CUDA;
    if (cudaEventRecord(p->hs_ev_in[slot], p->hs_in) != cudaSuccess) return ACTORQ_ERR_CUDA;
    if (cudaStreamWaitEvent(st, p->hs_ev_in[slot], 0) != cudaSuccess) return ACTORQ_ERR_CUDA;
    rc = forward_impl(p, p->hs_obs[slot], n, p->hs_out[slot], want_actions ? p->hs_act[slot] : nullptr, -1, nullptr, nullptr, st);
    if (rc != ACTORQ_OK) return rc;
    launches += p->launches;
    if (cudaEventRecord(p->hs_ev_comp[slot], st) != cudaSuccess) return ACTORQ_ERR_CUDA;
    if (cudaStreamWaitEvent(p->hs_outs, p->hs_ev_comp[slot], 0) != cudaSuccess) return ACTORQ_ERR_CUDA;
    if (cudaMemcpyAsync((char *)out_host + (size_t)r0 * out_row, p->hs_out[slot], (size_t)n * out_row,
                        cudaMemcpyDeviceToHost, p->hs_outs) != cudaSuccess) return ACTORQ_ERR_CUDA;
    if (want_actions &&
        cudaMemcpyAsync(actions_host + r0, p->hs_act[slot], (size_t)n * sizeof(int), cudaMemcpyDeviceToHost, p->hs_outs) != cudaSuccess)
      return ACTORQ_ERR_CUDA;
    if (cudaEventRecord(p->hs_ev_out[slot], p->hs_outs) != cudaSuccess) return ACTORQ_ERR_CUDA;
    done += n;
  }
  // the call is complete, for the caller's stream, when the last copies out are
  for (int i = 0; i < S && i < n_chunks; ++i)
    if (cudaStreamWaitEvent(st, p->hs_ev_out[i], 0) != cudaSuccess) return ACTORQ_ERR_CUDA;
  p->launches = launches;
  return ACTORQ_OK;
}

void actorq_free(actorq_policy *p) {
  if (!p) return;
  cudaDeviceSynchronize();
  if (p->hs_ready) {
    cudaStreamDestroy(p->hs_in);
    cudaStreamDestroy(p->hs_outs);
    for (int i = 0; i < actorq_policy::kHostSlots; ++i) {
      cudaEventDestroy(p->hs_ev_in[i]); cudaEventDestroy(p->hs_ev_comp[i]); cudaEventDestroy(p->hs_ev_out[i]);
    }
  }
  if (p->hs_mem) cudaFree(p->hs_mem);
  if (p->scratch[0]) cudaFree(p->scratch[0]);
  if (p->fcp_mem) cudaFree(p->fcp_mem);
  if (p->f16_act) cudaFree(p->f16_act);
  if (p->f16_pool) cudaFree(p->f16_pool);
  if (p->pool) cudaFree(p->pool);
  cudaGetLastError();
  delete p;
}

int actorq_policy_export_layer_channels(actorq_policy *p, int layer, signed char *w_q, float *scales, int *zero_points,
                                        void *cuda_stream) {
  if (p && p->precision == 16) return ACTORQ_ERR_UNSUPPORTED;      // int8 policies only
  if (!p || layer < 0 || layer >= p->n_layers || !w_q || !scales || !zero_points) return ACTORQ_ERR_INVALID_ARG;
  const LayerDev &L = p->layers[layer];
  if (!L.g.per_channel) return ACTORQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaMemcpyAsync(w_q, L.wq, (size_t)L.g.w_elems, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return ACTORQ_ERR_CUDA;
  if (cudaMemcpyAsync(scales, L.ch_sw, sizeof(float) * L.g.N, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ACTORQ_ERR_CUDA;
  if (cudaMemcpyAsync(zero_points, L.ch_zw, sizeof(int) * L.g.N, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ACTORQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return ACTORQ_ERR_CUDA;
  return ACTORQ_OK;
}

int actorq_policy_export_layer(actorq_policy *p, int layer, signed char *w_q, float *scale, int *zero_point,
                               void *cuda_stream) {
  if (p && p->precision == 16) return ACTORQ_ERR_UNSUPPORTED;      // int8 policies only
  if (!p || layer < 0 || layer >= p->n_layers || !w_q || !scale || !zero_point) return ACTORQ_ERR_INVALID_ARG;
  if (p->layers[layer].g.per_channel) return ACTORQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  LayerParams lp;
  if (cudaMemcpyAsync(w_q, p->layers[layer].wq, (size_t)p->layers[layer].g.w_elems, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return ACTORQ_ERR_CUDA;
  if (cudaMemcpyAsync(&lp, p->d_params + layer, sizeof(lp), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return ACTORQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return ACTORQ_ERR_CUDA;
  *scale = lp.s_w;
  *zero_point = lp.z_w;
  return ACTORQ_OK;
}

int actorq_policy_last_device_status(actorq_policy *p) {
  if (!p) return ACTORQ_ERR_INVALID_ARG;
  int st = 0;
  if (cudaMemcpy(&st, p->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return ACTORQ_ERR_CUDA;
  if (st != 0 && cudaMemset(p->d_status, 0, sizeof(int)) != cudaSuccess) return ACTORQ_ERR_CUDA;
  return st;
}

int actorq_policy_timeout_info(actorq_policy *p, int *info8) {
  if (!p || !info8) return ACTORQ_ERR_INVALID_ARG;
  int w[8];
  if (cudaMemcpy(w, p->d_status, sizeof(w), cudaMemcpyDeviceToHost) != cudaSuccess) return ACTORQ_ERR_CUDA;
  // reported, block, warp, barrier offset inside the kernel's barrier block, phase parity
  info8[0] = w[1]; info8[1] = w[2]; info8[2] = w[3]; info8[3] = w[1] ? w[4] - w[7] : 0; info8[4] = w[5];
  info8[5] = info8[6] = info8[7] = 0;
  if (w[1] != 0 && cudaMemset(p->d_status + 1, 0, sizeof(int) * 5) != cudaSuccess) return ACTORQ_ERR_CUDA;
  return ACTORQ_OK;
}

int actorq_policy_blob_bytes(const actorq_policy *p, long long *bytes) {
  if (p && p->precision == 16) return ACTORQ_ERR_UNSUPPORTED;
  if (!p || !bytes) return ACTORQ_ERR_INVALID_ARG;
  *bytes = blob_bytes(p);
  return ACTORQ_OK;
}

int actorq_policy_export_blob(actorq_policy *p, void *blob, long long capacity, void *cuda_stream) {
  if (p && p->precision == 16) return ACTORQ_ERR_UNSUPPORTED;      // int8 policies only
  if (!p || !blob) return ACTORQ_ERR_INVALID_ARG;
  if (capacity < blob_bytes(p) || (reinterpret_cast<uintptr_t>(blob) & 15) != 0) return ACTORQ_ERR_INVALID_ARG;
  return launch_export_blob(p, blob, (cudaStream_t)cuda_stream);
}

int actorq_policy_import_blob(actorq_policy *p, const void *blob, long long bytes, void *cuda_stream) {
  if (p && p->precision == 16) return ACTORQ_ERR_UNSUPPORTED;      // int8 policies only
  if (!p || !blob) return ACTORQ_ERR_INVALID_ARG;
  if (bytes != blob_bytes(p) || (reinterpret_cast<uintptr_t>(blob) & 15) != 0) return ACTORQ_ERR_INVALID_ARG;
  return launch_import_blob(p, blob, (cudaStream_t)cuda_stream);
}

int actorq_policy_set_fused_variant(actorq_policy *p, int variant) {
  if (p && p->precision == 16) return ACTORQ_ERR_UNSUPPORTED;      // int8 policies only
  if (!p || variant < 0 || variant > 4) return ACTORQ_ERR_INVALID_ARG;
  if (variant == 3) {
    if (!p->fcp_ok) return ACTORQ_ERR_UNSUPPORTED;
    p->fused_variant = variant;
    return ACTORQ_OK;
  }
  if (variant != 0 && !p->fused_ok) return ACTORQ_ERR_UNSUPPORTED;
  if (variant == 2 && !actorq::fused_pair_supported(p)) return ACTORQ_ERR_UNSUPPORTED;
  if (variant == 4 && !actorq::fused_resident_supported(p)) return ACTORQ_ERR_UNSUPPORTED;
  p->fused_variant = variant;
  return ACTORQ_OK;
}

int actorq_selftest_bounded_wait(actorq_policy *p, long long limit_ns, void *cuda_stream) {
  if (!p) return ACTORQ_ERR_INVALID_ARG;
  return launch_selftest_bounded_wait(p, limit_ns, (cudaStream_t)cuda_stream);
}

int actorq_selftest_int8_mma_peak(actorq_policy *p, long long mma_groups, int a_in_tmem, long long *ops, void *cuda_stream) {
  if (!p || mma_groups < 1 || mma_groups > (1ll << 24)) return ACTORQ_ERR_INVALID_ARG;
  return launch_selftest_int8_mma_peak(p, mma_groups, a_in_tmem != 0, ops, (cudaStream_t)cuda_stream);
}

int actorq_policy_last_launch_count(const actorq_policy *p) { return p ? p->launches : 0; }

const char *actorq_version(void) { return "actorq-b200 0.1 sm_100a"; }

}  // extern "C"
