// The fp16 actor (paper Section 3.2: policies are quantized "to fp16 and int8"; the q = 16 rows of the
// communication-vs-computation study): the learner's fp32 policy is CAST to binary16 at a broadcast
// instead of quantized to int8, and inference runs with binary16 operands and binary32 accumulation.
//   layer:  y[n] = sum_k a[k] w[n][k] + b[n]     a, w binary16 (round to nearest even), b binary32
//   hidden: a_next = rn16(max(y, 0));   last: out = tanh(y) or y, greedy action = lowest index of the maximum
// One launch per layer on CTA pairs, the structure of the int8 layer kernel (fc_pair.cu) with
// tcgen05.mma.cta_group::2.kind::f16: work item = tile pair (256 rows) x 256 output columns; warp 0
// streams, per 128-byte K block (64 elements), the CTA's 16 KB block of A and its half of the 256
// weight rows into a 6-stage ring (bulk copies, this GPU's memory, no multicast); warp 1 issues four
// K = 16 MMAs per block (even CTA) or relays "my half has landed" (odd CTA); warps 2-9 drain one of
// the two alternating 256-column binary32 accumulators, add the bias, apply ReLU, round to binary16
// and write 16-byte pieces of the next layer's operand blocks.  Activations between layers live in
// device memory as operand blocks ([128 rows][128 B], 128-byte swizzle).  Every wait is bounded.
#include <new>
#include <cuda_fp16.h>
#include "tcgen05.cuh"

namespace actorq {
namespace f16 {

constexpr int kEpiWarp0 = 2;
constexpr int kEpiWarps = 8;           // two per lane quarter: 128 of a chunk's 256 columns each
constexpr int kThreads = (kEpiWarp0 + kEpiWarps) * 32;
constexpr int kAccCols = 256;
constexpr int kStage = 2 * kStageBytes;    // A block + this CTA's half of the B block
constexpr int kMaxStages = 6;
constexpr int kBlockK = 64;            // binary16 elements per 128-byte K block

struct Args {
  const uint8_t *a_img;    // input operand blocks  [tile][nkb][16 KB]
  uint8_t *out_img;        // output operand blocks [tile][nkb_out][16 KB] (hidden layers)
  const uint8_t *w_img;    // weight image [128-row tile][nkb][16 KB]
  const float *bias;       // [N padded to 128], zeros for a layer without bias
  int K, N, Npad, nkb, nchunk, nkb_out;
  int last, head;
  long long batch, n_tile_pairs, n_items;
  float *out;
  int *actions;
  int n_stages;
  int *status;
};

struct __align__(16) Barriers {
  uint64_t ring_full[kMaxStages];
  uint64_t ring_empty[kMaxStages];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

// instruction descriptor: D = F32, A = B = F16, both K-major, M = 256 (the pair), n columns
__device__ __forceinline__ uint32_t instr_desc_f16_pair(int n) {
  return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}
__device__ __forceinline__ void mma2_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// fp32 weights [N][K] -> binary16 weight image: tile (n / 128, k / 64) of 16 KB, row n % 128 of 128
// bytes, the 16-byte piece index XOR-ed with (row % 8); everything outside N x K stays zero
__global__ void cast_weights_kernel(const float *__restrict__ w, int N, int K, int nkb, uint8_t *__restrict__ img) {
  const long long total = (long long)N * K;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(i / K), k = (int)(i - (long long)n * K);
    const uint32_t r = (uint32_t)n & 127u, kk = (uint32_t)k & 63u;
    const size_t off = (((size_t)(n >> 7) * nkb + (size_t)(k >> 6)) << 14) + (r << 7) + ((((kk >> 3) ^ (r & 7u))) << 4) + ((kk & 7u) << 1);
    *reinterpret_cast<__half *>(img + off) = __float2half_rn(__ldg(w + i));
  }
}
__global__ void copy_bias_kernel(const float *__restrict__ b, int N, float *__restrict__ dst) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) dst[i] = b ? __ldg(b + i) : 0.0f;
}
// fp32 observations [batch][K] -> binary16 operand blocks; rows >= batch and columns >= K are zeros
__global__ void cast_obs_kernel(const float *__restrict__ x, long long batch, long long rows_pad, int K, int nkb, uint8_t *__restrict__ img) {
  const long long total = rows_pad * (long long)(nkb * kBlockK);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long row = i / (nkb * kBlockK);
    const int k = (int)(i - row * (nkb * kBlockK));
    const float v = (row < batch && k < K) ? __ldg(x + row * K + k) : 0.0f;
    const uint32_t r = (uint32_t)(row & 127), kk = (uint32_t)k & 63u;
    const size_t off = ((((size_t)(row >> 7)) * nkb + (size_t)(k >> 6)) << 14) + (r << 7) + ((((kk >> 3) ^ (r & 7u))) << 4) + ((kk & 7u) << 1);
    *reinterpret_cast<__half *>(img + off) = __float2half_rn(v);
  }
}

__global__ void __launch_bounds__(kThreads, 1)
fp16_pair_kernel(const __grid_constant__ Args A) {
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {      // (the same in both CTAs of a pair, so both leave)
    if (threadIdx.x == 0) atomicMax(A.status, (int)ACTORQ_ERR_CUDA);
    return;
  }
  uint8_t *ring = smem;
  Barriers *bars = reinterpret_cast<Barriers *>(ring + A.n_stages * kStage);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const long long pair_idx = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  volatile int *abort_flag = &bars->abort_flag;
  const uint32_t peer_abort = mapa_u32(smem_u32(&bars->abort_flag), rank ^ 1u);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(&bars->ring_full[s], rank == 0 ? 2 : 1);    // own bulk copies (+ the odd CTA's relay)
      mbar_init(&bars->ring_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->acc_full[b], 1);
      mbar_init(&bars->acc_empty[b], 2 * kEpiWarps);
    }
    mbar_init(&bars->drain, 1);
    bars->abort_flag = 0;
    if (blockIdx.x == 0) A.status[7] = (int)smem_u32(bars);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(&bars->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();        // both CTAs' barriers exist before anyone arrives remotely
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  // programmatic dependent launch: nothing below runs before the previous kernel (the cast, or the
  // layer before) has completed
  griddep_launch_dependents();
  griddep_wait();

  if (warp == 0) {
    // ---------------- producer: this CTA's A block and its half of the weight rows, per K block ----------------
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    for (long long item = pair_idx; item < A.n_items && ok; item += n_pairs) {
      const long long tp = item / A.nchunk;
      const int c = (int)(item - tp * A.nchunk);
      const long long tile = 2 * tp + rank;
      const int rows_c = min(kAccCols, A.Npad - c * kAccCols);
      const int half_rows = rows_c >> 1;
      const int n_first = c * kAccCols + (int)rank * half_rows;     // weight rows [n_first, + half_rows)
      const int t0 = n_first >> 7, r0 = n_first & 127;
      const int rows_a = min(half_rows, 128 - r0);                  // rows taken from image tile t0
      const int rows_b = half_rows - rows_a;                        // the rest, from the next tile
      const uint32_t bytes = (uint32_t)kStageBytes + (uint32_t)half_rows * 128;
      for (int kb = 0; kb < A.nkb; ++kb) {
        ok = mbar_wait_warp(&bars->ring_empty[s], ph ^ 1, abort_flag, A.status);
        if (!ok) break;
        if (elect_one()) {
          uint8_t *dst = ring + s * kStage;
          mbar_expect_tx(&bars->ring_full[s], bytes);
          bulk_g2s(dst, A.a_img + (((size_t)tile * A.nkb + kb) << 14), (uint32_t)kStageBytes, &bars->ring_full[s]);
          bulk_g2s(dst + kStageBytes, A.w_img + (((size_t)t0 * A.nkb + kb) << 14) + ((size_t)r0 << 7), (uint32_t)rows_a * 128,
                   &bars->ring_full[s]);
          if (rows_b > 0)
            bulk_g2s(dst + kStageBytes + rows_a * 128, A.w_img + (((size_t)(t0 + 1) * A.nkb + kb) << 14), (uint32_t)rows_b * 128,
                     &bars->ring_full[s]);
        }
        __syncwarp();
        if (++s == A.n_stages) { s = 0; ph ^= 1; }
      }
    }
    if (!ok) for (int i = 0; i < 64; ++i) __nanosleep(1000);      // bulk copies still in flight into this CTA
  } else if (warp == 1 && rank == 0) {
    // ---------------- MMA issuer (even CTA) ----------------
    int s = 0;
    uint32_t ph = 0, it = 0;
    const uint32_t ring_base = smem_u32(ring);
    bool ok = true;
    for (long long item = pair_idx; item < A.n_items && ok; item += n_pairs, ++it) {
      const int c = (int)(item % A.nchunk);
      const int rows_c = min(kAccCols, A.Npad - c * kAccCols);
      const uint32_t idesc = instr_desc_f16_pair(rows_c);
      const uint32_t buf = it & 1, use = it >> 1;
      const uint32_t d_tmem = tmem + buf * kAccCols;
      ok = mbar_wait_warp_cl(&bars->acc_empty[buf], (use & 1) ^ 1, abort_flag, peer_abort, A.status);
      if (!ok) break;
      tc_fence_after();
      for (int kb = 0; kb < A.nkb; ++kb) {
        ok = mbar_wait_warp_cl(&bars->ring_full[s], ph, abort_flag, peer_abort, A.status);
        if (!ok) break;
        tc_fence_after();
        const int ksteps = (min(kBlockK, A.K - kb * kBlockK) + 15) >> 4;        // K = 16 elements (32 bytes) per instruction
        const uint64_t adesc = ((uint64_t)kDescHi << 32) | desc_lo(ring_base + s * kStage);
        const uint64_t bdesc = ((uint64_t)kDescHi << 32) | desc_lo(ring_base + s * kStage + kStageBytes);
        if (elect_one()) {
          for (int ks = 0; ks < ksteps; ++ks)
            mma2_f16(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), idesc, (kb | ks) != 0);
          mma_commit_pair(&bars->ring_empty[s], 3);
          if (kb + 1 == A.nkb) mma_commit_pair(&bars->acc_full[buf], 3);
        }
        __syncwarp();
        if (++s == A.n_stages) { s = 0; ph ^= 1; }
      }
    }
    // no MMA of this thread may still be running (in either CTA) when tensor memory is given back
    if (elect_one()) mma_commit_pair(&bars->drain, 1);
    __syncwarp();
    volatile int never = 0;
    mbar_wait_warp(&bars->drain, 0, &never, A.status);
  } else if (warp == 1) {
    // ---------------- relay (odd CTA): "my part of ring stage s has landed" -> even CTA ----------------
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    const uint32_t full0 = mapa_u32(smem_u32(&bars->ring_full[0]), 0);
    for (long long item = pair_idx; item < A.n_items && ok; item += n_pairs) {
      for (int kb = 0; kb < A.nkb; ++kb) {
        ok = mbar_wait_warp(&bars->ring_full[s], ph, abort_flag, A.status);
        if (!ok) break;
        if (lane == 0) mbar_arrive_cluster(full0 + 8u * (uint32_t)s);
        __syncwarp();
        if (++s == A.n_stages) { s = 0; ph ^= 1; }
      }
    }
  } else {
    // ---------------- epilogue (warps 2..9) ----------------
    const int ew = warp - kEpiWarp0;
    const int quarter = warp & 3;              // TMEM lanes this warp may touch: 32*quarter .. +31
    const int part = ew >> 2;                  // which 128 columns of the 256-column accumulator
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t acc_empty_leader = mapa_u32(smem_u32(&bars->acc_empty[0]), 0);
    uint32_t it = 0;
    bool ok = true;
    for (long long item = pair_idx; item < A.n_items && ok; item += n_pairs, ++it) {
      const long long tp = item / A.nchunk;
      const int c = (int)(item - tp * A.nchunk);
      const long long tile = 2 * tp + rank;
      const long long grow = tile * kTileM + row;
      const bool row_valid = grow < A.batch;
      const int rows_c = min(kAccCols, A.Npad - c * kAccCols);
      const uint32_t buf = it & 1, use = it >> 1;
      const uint32_t acc = tmem + lane_addr + buf * kAccCols;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_full[buf], use & 1, abort_flag, A.status));
      if (!ok) break;
      tc_fence_after();
      // this warp's 32-column slices of the chunk: hidden layers split the columns between the two
      // warps of a quarter; the head (at most 128 columns, whole rows for the greedy action) is done by part 0
      const int col_begin = A.last ? 0 : part * 128;
      const int col_end = A.last ? (part == 0 ? rows_c : 0) : min(rows_c, part * 128 + 128);
      const int n_slices = col_end > col_begin ? (col_end - col_begin + 31) / 32 : 0;
      if (n_slices == 0) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8u * buf);
      }
      float best_v = 0.0f;
      int best_n = -1;
      for (int sl = 0; sl < n_slices; ++sl) {
        const int col0 = col_begin + sl * 32;
        uint32_t r[32];
        tmem_ld32_wait(acc + col0, r);
        if (sl + 1 == n_slices) {              // the accumulator goes back to the issuer
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8u * buf);
        }
        const int n0 = c * kAccCols + col0;
        float v[32];
#pragma unroll
        for (int j4 = 0; j4 < 8; ++j4) {
          const float4 b4 = __ldg(reinterpret_cast<const float4 *>(A.bias + n0) + j4);
          v[4 * j4 + 0] = __fadd_rn(__uint_as_float(r[4 * j4 + 0]), b4.x);
          v[4 * j4 + 1] = __fadd_rn(__uint_as_float(r[4 * j4 + 1]), b4.y);
          v[4 * j4 + 2] = __fadd_rn(__uint_as_float(r[4 * j4 + 2]), b4.z);
          v[4 * j4 + 3] = __fadd_rn(__uint_as_float(r[4 * j4 + 3]), b4.w);
        }
        if (!A.last) {
          // ReLU, round to binary16, columns >= N are the next layer's K padding (zeros)
          uint32_t packed[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float lo = (n0 + 2 * j < A.N) ? fmaxf(v[2 * j], 0.0f) : 0.0f;
            const float hi = (n0 + 2 * j + 1 < A.N) ? fmaxf(v[2 * j + 1], 0.0f) : 0.0f;
            const __half2 h = __floats2half2_rn(lo, hi);
            packed[j] = *reinterpret_cast<const uint32_t *>(&h);
          }
          // 32 columns = 64 bytes = four 16-byte pieces of K block n0 / 64 of the next layer's operand row
          uint8_t *rowp = A.out_img + (((size_t)tile * A.nkb_out + (size_t)(n0 >> 6)) << 14) + ((uint32_t)row << 7);
          const uint32_t p0 = ((uint32_t)n0 & 63u) >> 3;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4 *>(rowp + (((p0 + q) ^ ((uint32_t)row & 7u)) << 4)) =
                make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
        } else {
          // (all 32 columns without branches, so that the tanh chains overlap; columns >= N never leave)
          if (A.head == ACTORQ_HEAD_ARGMAX) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (n0 + j < A.N && (v[j] > best_v || best_n < 0)) { best_v = v[j]; best_n = n0 + j; }
          } else if (A.head == ACTORQ_HEAD_TANH) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = tanhf(v[j]);
          }
          if (row_valid) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (n0 + j < A.N) A.out[grow * A.N + n0 + j] = v[j];
          }
        }
      }
      if (A.last && A.head == ACTORQ_HEAD_ARGMAX && part == 0 && row_valid) A.actions[grow] = best_n;
    }
  }

  // teardown: every role of both CTAs arrives here (aborted or not); no remote arrive, commit or MMA
  // may target a CTA that has already left, and tensor memory goes back before the CTAs exit
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, 512);
  }
}

}  // namespace f16

// ---- host side ------------------------------------------------------------------------------

static int f16_round_up(int v, int m) { return (v + m - 1) / m * m; }
static size_t f16_align(size_t v) { return (v + 1023) & ~(size_t)1023; }

bool fp16_supported(const actorq_policy *p) {
  if (p->obs_dtype != ACTORQ_OBS_F32) return false;
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerGeom &g = p->layers[l].g;
    const bool last = (l + 1 == p->n_layers);
    if (g.kind != ACTORQ_FC || g.per_channel) return false;
    if (g.K > 8192 || (last ? g.N > 128 : g.N > 8192)) return false;
  }
  return true;
}

// one pool: status block, then per layer the binary16 weight image and the binary32 bias
int fp16_setup(actorq_policy *p) {
  size_t off = f16_align(sizeof(int) * 16);
  size_t o_img[ACTORQ_MAX_LAYERS], o_bias[ACTORQ_MAX_LAYERS];
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerGeom &g = p->layers[l].g;
    const size_t img = (size_t)((g.N + 127) / 128) * (size_t)((g.K + f16::kBlockK - 1) / f16::kBlockK) * kStageBytes;
    o_img[l] = off; off = f16_align(off + img);
    o_bias[l] = off; off = f16_align(off + sizeof(float) * (size_t)f16_round_up(g.N, 128));
  }
  if (cudaMalloc(&p->f16_pool, off) != cudaSuccess) { cudaGetLastError(); p->f16_pool = nullptr; return ACTORQ_ERR_NOMEM; }
  if (cudaMemset(p->f16_pool, 0, off) != cudaSuccess) return ACTORQ_ERR_CUDA;
  char *base = (char *)p->f16_pool;
  p->d_status = (int *)base;
  for (int l = 0; l < p->n_layers; ++l) {
    p->f16_img[l] = (uint8_t *)(base + o_img[l]);
    p->f16_bias[l] = (float *)(base + o_bias[l]);
  }
  return ACTORQ_OK;
}

// the cast at a broadcast: fp32 weights -> binary16 images, biases copied; no allocation, no host synchronisation
int launch_cast_fp16(actorq_policy *p, cudaStream_t st) {
  p->launches = 0;
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerGeom &g = p->layers[l].g;
    const long long total = (long long)g.N * g.K;
    long long blocks = (total + 255) / 256;
    if (blocks > (long long)p->sm_count * 16) blocks = (long long)p->sm_count * 16;
    f16::cast_weights_kernel<<<(unsigned)blocks, 256, 0, st>>>(p->layers[l].w_f32, g.N, g.K, (g.K + f16::kBlockK - 1) / f16::kBlockK, p->f16_img[l]);
    f16::copy_bias_kernel<<<(g.N + 255) / 256, 256, 0, st>>>(p->layers[l].b_f32, g.N, p->f16_bias[l]);
    p->launches += 2;
  }
  return cuda_ok(cudaGetLastError());
}

int launch_forward_fp16(actorq_policy *p, const void *obs, long long batch, float *out, int *actions, cudaStream_t st) {
  static bool attr_set[64] = {false};
  static int max_clusters[64] = {0};
  const int dev = p->device;
  if (dev < 0 || dev >= 64) return ACTORQ_ERR_UNSUPPORTED;
  const int n_stages = f16::kMaxStages;
  const int smem_bytes = n_stages * f16::kStage + (int)sizeof(f16::Barriers);
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.blockDim = dim3(f16::kThreads);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(f16::fp16_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess) return ACTORQ_ERR_CUDA;
    cfg.gridDim = dim3((unsigned)(p->sm_count & ~1));
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, f16::fp16_pair_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
    max_clusters[dev] = n;
    attr_set[dev] = true;
  }
  if (max_clusters[dev] < 1) return ACTORQ_ERR_UNSUPPORTED;
  const long long n_tiles = (batch + kTileM - 1) / kTileM;
  const long long n_tile_pairs = (n_tiles + 1) / 2;
  const long long rows_pad = n_tile_pairs * 2 * kTileM;
  // two activation buffers of rows_pad x (widest layer input, in whole 128-byte K blocks) binary16 values
  int kmax = 0;
  for (int l = 0; l < p->n_layers; ++l) kmax = p->layers[l].g.K > kmax ? p->layers[l].g.K : kmax;
  const size_t one = (size_t)rows_pad * (size_t)f16_round_up(kmax, f16::kBlockK) * 2;
  if (rows_pad > p->f16_rows) {
    if (p->f16_act) cudaFree(p->f16_act);
    p->f16_act = nullptr;
    p->f16_rows = 0;
    if (cudaMalloc(&p->f16_act, 2 * one) != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_NOMEM; }
    p->f16_rows = rows_pad;
  }
  const size_t stride = (size_t)p->f16_rows * (size_t)f16_round_up(kmax, f16::kBlockK) * 2;
  uint8_t *bufs[2] = {(uint8_t *)p->f16_act, (uint8_t *)p->f16_act + stride};
  {
    const LayerGeom &g0 = p->layers[0].g;
    const int nkb0 = (g0.K + f16::kBlockK - 1) / f16::kBlockK;
    const long long total = rows_pad * (long long)(nkb0 * f16::kBlockK);
    long long blocks = (total + 255) / 256;
    if (blocks > (long long)p->sm_count * 32) blocks = (long long)p->sm_count * 32;
    f16::cast_obs_kernel<<<(unsigned)blocks, 256, 0, st>>>((const float *)obs, batch, rows_pad, g0.K, nkb0, bufs[0]);
    p->launches++;
  }
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerGeom &g = p->layers[l].g;
    const bool last = (l + 1 == p->n_layers);
    f16::Args A;
    memset(&A, 0, sizeof(A));
    A.a_img = bufs[l & 1];
    A.out_img = last ? nullptr : bufs[(l + 1) & 1];
    A.w_img = p->f16_img[l];
    A.bias = p->f16_bias[l];
    A.K = g.K; A.N = g.N; A.Npad = f16_round_up(g.N, 32);
    A.nkb = (g.K + f16::kBlockK - 1) / f16::kBlockK;
    A.nchunk = (A.Npad + f16::kAccCols - 1) / f16::kAccCols;
    A.nkb_out = (g.N + f16::kBlockK - 1) / f16::kBlockK;
    A.last = last ? 1 : 0;
    A.head = p->head;
    A.batch = batch;
    A.n_tile_pairs = n_tile_pairs;
    A.n_items = n_tile_pairs * A.nchunk;
    A.out = out;
    A.actions = actions;
    A.n_stages = n_stages;
    A.status = p->d_status;
    const long long pairs = A.n_items < max_clusters[dev] ? A.n_items : max_clusters[dev];
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, f16::fp16_pair_kernel, A);
    p->launches++;
    if (e != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_CUDA; }
  }
  return ACTORQ_OK;
}

}  // namespace actorq
