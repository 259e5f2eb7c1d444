// Bare int8 tensor-core loop: the achieved dense INT8 rate of this GPU, measured with the same
// instruction the layer kernels use (tcgen05.mma.cta_group::2.kind::i8, M = 256, n = 256, K = 32 per
// instruction, both operands resident, no epilogue, no data movement).  It is the denominator the
// benchmark reports tensor-bound fractions against; it computes nothing of the paper's method.
//
// One cluster of two CTAs per SM pair.  Each CTA holds one 128-row x 128-byte A block and its half
// (128 rows) of a 256-row B block in shared memory, filled with pseudo-random bytes (all-zero
// operands would draw less power and flatter the clock).  One thread of the even CTA issues `groups`
// groups of four MMAs (one 128-byte K block each), alternating between two 256-column accumulators,
// then commits and waits (bounded) for the tensor cores to drain.
#include "tcgen05.cuh"

namespace actorq {
namespace peak {

constexpr int kThreads = 128;
constexpr int kSmemBytes = 160 * 1024;      // more than half an SM's shared memory: one CTA per SM

struct __align__(16) Bars {
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(kThreads, 1)
int8_mma_peak_kernel(long long groups, int a_in_tmem, int *status) {
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicMax(status, (int)ACTORQ_ERR_CUDA);
    return;
  }
  uint8_t *a_blk = smem;                       // 16 KB
  uint8_t *b_blk = smem + kStageBytes;         // 16 KB
  Bars *bars = reinterpret_cast<Bars *>(smem + 2 * kStageBytes);
  const int warp = threadIdx.x >> 5;
  const uint32_t rank = cluster_ctarank();

  // operand bytes: an integer hash of the position (any values do; the accumulators are never read)
  uint32_t *words = reinterpret_cast<uint32_t *>(smem);
  for (int i = threadIdx.x; i < 2 * kStageBytes / 4; i += kThreads) {
    uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 40503u;
    h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
    words[i] = h;
  }
  fence_proxy_async();
  if (threadIdx.x == 0) {
    mbar_init(&bars->drain, 1);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(&bars->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (a_in_tmem) {     // the A block as 32 tensor-memory columns (4 codes per column), lanes = rows
    uint32_t v[8];
    for (int c = 0; c < 32; c += 8) {
      for (int j = 0; j < 8; ++j) v[j] = words[(threadIdx.x * 32 + c + j) & 4095];
      tmem_st8(tmem + ((uint32_t)(warp * 32) << 16) + 256 + c, v);
    }
    tmem_wait_st();
    tc_fence_before();
  }
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();

  if (warp == 1 && rank == 0) {
    const uint32_t idesc = instr_desc_pair(256, false);
    const uint32_t a_lo = desc_lo(smem_u32(a_blk)), b_lo = desc_lo(smem_u32(b_blk));
    if (elect_one()) {
      for (long long g = 0; g < groups; ++g) {
        const uint32_t fresh = ((g & 127) < 2) ? 0u : 1u;          // restart the sums now and then
        if (a_in_tmem) mma2x4_i8_ts(tmem, tmem + 256, b_lo, kDescHi, idesc, fresh);
        else mma2x4_i8_ss(tmem + (uint32_t)(g & 1) * 256u, a_lo, b_lo, kDescHi, idesc, fresh);
      }
      mma_commit_pair(&bars->drain, 1);
    }
    __syncwarp();
    mbar_wait_warp(&bars->drain, 0, &bars->abort_flag, status);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, 512);
  }
}

}  // namespace peak

int launch_selftest_int8_mma_peak(actorq_policy *p, long long groups, int a_in_tmem, long long *ops, cudaStream_t st) {
  static bool attr_set[64] = {false};
  static int max_clusters[64] = {0};
  const int dev = p->device;
  if (dev < 0 || dev >= 64) return ACTORQ_ERR_UNSUPPORTED;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(peak::kThreads);
  cfg.dynamicSmemBytes = (size_t)peak::kSmemBytes;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(peak::int8_mma_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, peak::kSmemBytes) != cudaSuccess)
      return ACTORQ_ERR_CUDA;
    cfg.gridDim = dim3((unsigned)(p->sm_count & ~1));
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, peak::int8_mma_peak_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
    max_clusters[dev] = n;
    attr_set[dev] = true;
  }
  int pairs = max_clusters[dev];
  if (pairs > p->sm_count / 2) pairs = p->sm_count / 2;
  if (pairs < 1) return ACTORQ_ERR_UNSUPPORTED;
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  // one instruction: M = 256 rows x n = 256 columns x K = 32, two operations per multiply-accumulate
  if (ops) *ops = (long long)pairs * groups * 4ll * (256ll * 256ll * 32ll * 2ll);
  const cudaError_t e = cudaLaunchKernelEx(&cfg, peak::int8_mma_peak_kernel, groups, a_in_tmem, p->d_status);
  if (e != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_CUDA; }
  return ACTORQ_OK;
}

}  // namespace actorq
