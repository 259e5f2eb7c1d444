// Layer-at-a-time int8 inference for architectures the fused tensor-core kernels do not cover
// (and the first, plainly written device statement of the arithmetic):
//   acc = sum_k (a_q - z_a)(w_q - z_w) + bias_q           int32, exact
//   hidden: a_next = clamp(rne((float)acc * M) + z_out, z_out, 127)
//   last:   y = (float)acc * P, then tanh / argmax         (paper Section 3.2, Eq. 3)
// Activations between layers are int8 codes in device scratch, [batch][features] with
// convolutional features in (c, h, w) order.
#include "common.cuh"
#include "explore_rng.cuh"

namespace actorq {

// q = clamp(rne(t) + z, lo_code, 127) evaluated as rne(clamp(t, lo_code - z, 127 - z)) + z:
// rounding is monotone and fixes integers, so clamping before or after it is the same.
__device__ __forceinline__ int round_clamp_code(float t, int z, int lo_code) {
  t = fminf(fmaxf(t, (float)(lo_code - z)), (float)(127 - z));
  return __float2int_rn(t) + z;
}

__global__ void quantize_obs_f32_kernel(const float *__restrict__ x, long long n,
                                        const LayerParams *__restrict__ params, int8_t *__restrict__ q) {
  const LayerParams p = params[0];
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    float t = __fmul_rn(__ldg(x + i), p.inv_s_a);
    if (t != t) t = 0.0f;                                  // NaN observation -> real 0
    q[i] = (int8_t)round_clamp_code(t, p.z_a, -128);
  }
}

__global__ void quantize_obs_u8_kernel(const uint8_t *__restrict__ u, long long n, int8_t *__restrict__ q) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    q[i] = (int8_t)((int)__ldg(u + i) - 128);
}

struct GenericLayerArgs {
  LayerGeom g;
  const int8_t *a;        // [batch][in_elems]
  const int8_t *wq;       // [N][K]
  const int *bias_q;      // [N]
  const int *ch_zw;       // per-channel layers: [N] weight zero-points, multipliers, accumulator units
  const float *ch_M;
  const float *ch_P;
  int8_t *a_next;         // [batch][out_elems] (hidden) or nullptr
  float *y;               // [batch][out_elems] (last) or nullptr
  int *dbg_acc;           // optional [batch][out_elems]
  int8_t *dbg_act;        // optional copy of a_next
  int apply_tanh;
  int layer;
  long long batch;
};

__device__ __forceinline__ void finish_output(const GenericLayerArgs &A, const LayerParams &p, long long idx, int n, int acc) {
  if (A.dbg_acc) A.dbg_acc[idx] = acc;
  if (A.a_next) {
    const float M = A.ch_M ? A.ch_M[n] : p.M;
    int q = round_clamp_code(__fmul_rn(__int2float_rn(acc), M), p.z_out, p.z_out);
    A.a_next[idx] = (int8_t)q;
    if (A.dbg_act) A.dbg_act[idx] = (int8_t)q;
  } else {
    const float P = A.ch_P ? A.ch_P[n] : p.P;
    float y = __fmul_rn(__int2float_rn(acc), P);
    A.y[idx] = A.apply_tanh ? tanhf(y) : y;
  }
}

__global__ void __launch_bounds__(256)
fc_generic_kernel(const GenericLayerArgs A, const LayerParams *__restrict__ params) {
  const LayerParams p = params[A.layer];
  const int K = A.g.K, N = A.g.N;
  const long long total = A.batch * N;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const long long b = idx / N;
    const int n = (int)(idx - b * N);
    const int8_t *__restrict__ a = A.a + b * K;
    const int8_t *__restrict__ w = A.wq + (long long)n * K;
    const int z_w = A.ch_zw ? A.ch_zw[n] : p.z_w;
    int acc = 0;
    for (int k = 0; k < K; ++k) acc += ((int)a[k] - p.z_a) * ((int)w[k] - z_w);
    finish_output(A, p, idx, n, acc + A.bias_q[n]);
  }
}

__global__ void __launch_bounds__(256)
conv_generic_kernel(const GenericLayerArgs A, const LayerParams *__restrict__ params) {
  const LayerParams p = params[A.layer];
  const LayerGeom &g = A.g;
  const long long total = A.batch * g.out_elems;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    long long t = idx;
    const int ow = (int)(t % g.out_w); t /= g.out_w;
    const int oh = (int)(t % g.out_h); t /= g.out_h;
    const int o = (int)(t % g.out_c);
    const long long b = t / g.out_c;
    const int8_t *__restrict__ a = A.a + b * g.in_elems;
    const int8_t *__restrict__ w = A.wq + (long long)o * g.K;
    const int z_w = A.ch_zw ? A.ch_zw[o] : p.z_w;
    int acc = 0;
    for (int c = 0; c < g.in_c; ++c)
      for (int kh = 0; kh < g.kh; ++kh) {
        const int8_t *arow = a + ((long long)c * g.in_h + (oh * g.stride + kh)) * g.in_w + ow * g.stride;
        const int8_t *wrow = w + (c * g.kh + kh) * g.kw;
        for (int kw = 0; kw < g.kw; ++kw) acc += ((int)arow[kw] - p.z_a) * ((int)wrow[kw] - z_w);
      }
    finish_output(A, p, idx, o, acc + A.bias_q[o]);
  }
}

// greedy action: lowest index of the row maximum
__global__ void argmax_kernel(const float *__restrict__ y, long long batch, int N, int *__restrict__ actions) {
  for (long long b = (long long)blockIdx.x * blockDim.x + threadIdx.x; b < batch; b += (long long)gridDim.x * blockDim.x) {
    const float *row = y + b * N;
    int best = 0;
    float bv = row[0];
    for (int n = 1; n < N; ++n) {
      float v = row[n];
      if (v > bv) { bv = v; best = n; }
    }
    actions[b] = best;
  }
}

// Exploration noise of the actors (the paper's D4PG set-up adds a Gaussian noise layer to the policy
// output, sigma per actor): two binary32 operations, then the clip that keeps the action in tanh's range.
__global__ void explore_kernel(float *__restrict__ out, const float *__restrict__ sigma, const float *__restrict__ noise,
                               long long batch, int out_dim) {
  const long long total = batch * out_dim;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const float v = __fadd_rn(out[i], __fmul_rn(__ldg(sigma + i / out_dim), __ldg(noise + i)));
    out[i] = fminf(fmaxf(v, -1.0f), 1.0f);
  }
}

static int grid_for(long long work, int threads, int sm_count) {
  long long blocks = (work + threads - 1) / threads;
  long long cap = (long long)sm_count * 32;
  return (int)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}

// the same with the draws of the counter-based generator (explore_rng.cuh), row = row0 + b
__global__ void explore_seeded_kernel(float *__restrict__ out, const float *__restrict__ sigma, uint32_t seed_lo, uint32_t seed_hi,
                                      long long row0, long long batch, int out_dim) {
  const long long total = batch * out_dim;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long b = i / out_dim;
    const int n = (int)(i - b * out_dim);
    const float z = exploration_normal(seed_lo, seed_hi, row0 + b, n);
    const float y = __fadd_rn(out[i], __fmul_rn(__ldg(sigma + b), z));
    out[i] = fminf(fmaxf(y, -1.0f), 1.0f);
  }
}

int launch_explore_seeded(float *out, const float *sigma, unsigned long long seed, long long row0, long long batch, int out_dim,
                          int sm_count, cudaStream_t st) {
  explore_seeded_kernel<<<grid_for(batch * out_dim, 256, sm_count), 256, 0, st>>>(out, sigma, (uint32_t)(seed & 0xffffffffull),
                                                                                 (uint32_t)(seed >> 32), row0, batch, out_dim);
  return cuda_ok(cudaGetLastError());
}

int launch_explore(float *out, const float *sigma, const float *noise, long long batch, int out_dim, int sm_count, cudaStream_t st) {
  explore_kernel<<<grid_for(batch * out_dim, 256, sm_count), 256, 0, st>>>(out, sigma, noise, batch, out_dim);
  return cuda_ok(cudaGetLastError());
}

// The layer-at-a-time forward with its two int8 activation buffers given by the caller: the policy's
// scratch (launch_forward_generic) or the fixed array of the allocation-free entry point.
static int run_generic_layers(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                              int dbg_layer, int *dbg_acc, int8_t *dbg_act, int8_t *cur, int8_t *nxt, cudaStream_t st) {
  const int sm = p->sm_count;
  const long long n0 = batch * p->layers[0].g.in_elems;
  if (p->obs_dtype == ACTORQ_OBS_U8_DIV255)
    quantize_obs_u8_kernel<<<grid_for(n0, 256, sm), 256, 0, st>>>((const uint8_t *)obs, n0, cur);
  else
    quantize_obs_f32_kernel<<<grid_for(n0, 256, sm), 256, 0, st>>>((const float *)obs, n0, p->d_params, cur);
  p->launches++;
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerDev &L = p->layers[l];
    const bool last = (l + 1 == p->n_layers);
    GenericLayerArgs A;
    A.g = L.g;
    A.a = cur;
    A.wq = L.wq;
    A.bias_q = L.bias_q;
    A.ch_zw = L.g.per_channel ? L.ch_zw : nullptr;
    A.ch_M = L.g.per_channel ? L.ch_M : nullptr;
    A.ch_P = L.g.per_channel ? L.ch_P : nullptr;
    A.a_next = last ? nullptr : nxt;
    A.y = last ? out : nullptr;
    A.dbg_acc = (l == dbg_layer) ? dbg_acc : nullptr;
    A.dbg_act = (l == dbg_layer && !last) ? dbg_act : nullptr;
    A.apply_tanh = (p->head == ACTORQ_HEAD_TANH);
    A.layer = l;
    A.batch = batch;
    const long long work = batch * L.g.out_elems;
    if (L.g.kind == ACTORQ_CONV2D)
      conv_generic_kernel<<<grid_for(work, 256, sm), 256, 0, st>>>(A, p->d_params);
    else
      fc_generic_kernel<<<grid_for(work, 256, sm), 256, 0, st>>>(A, p->d_params);
    p->launches++;
    int8_t *t = cur; cur = nxt; nxt = t;
  }
  if (p->head == ACTORQ_HEAD_ARGMAX) {
    argmax_kernel<<<grid_for(batch, 128, sm), 128, 0, st>>>(out, batch, p->layers[p->n_layers - 1].g.N, actions);
    p->launches++;
  }
  return cuda_ok(cudaGetLastError());
}

int launch_forward_generic(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                           int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st) {
  return run_generic_layers(p, obs, batch, out, actions, dbg_layer, dbg_acc, dbg_act, p->scratch[0], p->scratch[1], st);
}

// ---- forward without any allocation -----------------------------------------------------------
// The layer-at-a-time forward above keeps its two int8 activation buffers in scratch that the
// policy grows with cudaMalloc.  The entry point below runs the same kernels with both buffers
// carved out of one fixed array that is part of the library image, for callers that must not
// allocate device memory.  Every CUDA device that loads the library holds these bytes until the
// process exits, so the limit is deliberately modest.
static __device__ __align__(256) unsigned char g_static_scratch[ACTORQ_NOALLOC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address; the
// address a kernel can use has to be asked for, once per device, with that device current.
static unsigned char *static_scratch_ptr[64];

static int static_scratch_address(int device, unsigned char **out) {
  if (device < 0 || device >= 64) return ACTORQ_ERR_UNSUPPORTED;
  if (static_scratch_ptr[device] == nullptr) {
    unsigned char *ptr = nullptr;
    if (cudaGetSymbolAddress((void **)&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return ACTORQ_ERR_CUDA;
    }
    static_scratch_ptr[device] = ptr;
  }
  *out = static_scratch_ptr[device];
  return ACTORQ_OK;
}

}  // namespace actorq

extern "C" int actorq_policy_forward_noalloc(actorq_policy *p, const void *obs, long long batch, float *out,
                                             int *actions, void *cuda_stream) {
  if (p && p->precision == 16) return ACTORQ_ERR_UNSUPPORTED;      // int8 policies only
  using namespace actorq;
  if (!p || batch < 0) return ACTORQ_ERR_INVALID_ARG;
  p->launches = 0;
  if (batch == 0) return ACTORQ_OK;
  if (!obs || !out) return ACTORQ_ERR_INVALID_ARG;
  if (p->head == ACTORQ_HEAD_ARGMAX && !actions) return ACTORQ_ERR_INVALID_ARG;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) return ACTORQ_ERR_CUDA;
  if (device != p->device) return ACTORQ_ERR_INVALID_ARG;

  // both activation buffers must fit in the fixed array
  long long per_row = 0;
  for (int l = 0; l < p->n_layers; ++l) {
    if (p->layers[l].g.in_elems > per_row) per_row = p->layers[l].g.in_elems;
    if (p->layers[l].g.out_elems > per_row) per_row = p->layers[l].g.out_elems;
  }
  const long long half = ACTORQ_NOALLOC_SCRATCH_BYTES / 2;
  if (batch > half / per_row) return ACTORQ_ERR_SCRATCH_LIMIT;

  unsigned char *base = nullptr;
  int rc = static_scratch_address(device, &base);
  if (rc != ACTORQ_OK) return rc;
  int8_t *cur = reinterpret_cast<int8_t *>(base);
  int8_t *nxt = reinterpret_cast<int8_t *>(base + half);

  // Nothing in the array has to start at zero: the input quantizer writes every element the first
  // layer reads, and each layer writes every element the next one reads.
  return run_generic_layers(p, obs, batch, out, actions, -1, nullptr, nullptr, cur, nxt, (cudaStream_t)cuda_stream);
}
