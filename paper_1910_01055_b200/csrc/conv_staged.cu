// Implicit-GEMM int8 convolution with the layer's INPUT staged in shared memory (sm_100a, tcgen05):
// the convolutional trunk of DQN-style policies (paper Section 3.2: the three-layer convolutional
// Atari policy; arithmetic as everywhere: int8 x int8 -> int32 accumulators, one binary32 multiply
// to requantize, ReLU as the lower clamp).
//
//   raw[m][n] = sum_k A[m][k] * W[n][k],   m = (sample, oh, ow),  n = output channel <= 128,
//                                          k = position inside the receptive field
// Every input byte of a convolution is used by (kernel / stride)^2 output pixels.  Here it leaves
// device memory / L2 once: a work item is a group of G consecutive samples, whose input (uint8 NCHW
// frames for the first layer, int8 NHWC codes after that) arrives as ONE bulk copy into a
// double-buffered staging area, and the A operand blocks are built from shared memory, a WARP per
// output pixel with the lanes spread over the receptive field:
//   first layer  (K order (c, kh, kw), kw = 8 bytes): lane = (c, kh), two 4-byte loads (an input row
//                segment of 8 pixels), neighbouring lanes combine into 16-byte pieces;
//   later layers (K order (kh, kw, c)): lane = 16 channels of one input pixel, one 16-byte load, and
//                a quarter-warp reads 128 contiguous bytes (one kh row of the receptive field);
// both free of systematic bank conflicts, and a warp writes 16-byte pieces of ONE operand row.  Where
// the receptive field of a row starts in the staged input is read from a table built once per launch
// (items all have the same geometry), so the gather is loads, shuffles and stores only.
// The row sums of the codes (for the weight zero-point term) come from the tensor cores: the
// resident weight image gets one extra row of ones (row N), so accumulator column N of a row IS the
// sum of its codes, exactly.  The layer's whole weight image stays resident in shared memory (its
// column constants too); tensor memory holds two accumulators, so gather, MMAs and epilogue of
// neighbouring tiles overlap.
// Warps: 0 bulk-copy producer, 1 MMA issuer, 2-9 gather, 10-17 epilogue (two sets of four, one per
// accumulator; a warp per TMEM lane quarter).
// Every wait is bounded (ACTORQ_ERR_TIMEOUT in the status word, all roles leave, TMEM is freed).
#include "tcgen05.cuh"

namespace actorq {
namespace cst {

constexpr int kThreads = 576;
constexpr int kGatherWarp0 = 2;
constexpr int kGatherWarps = 8;        // (a multiple of 8: a warp's rows, kGatherWarps apart, share row & 7, the swizzle phase)
constexpr int kRowsWarp = kTileM / kGatherWarps;        // a warp's rows of a tile, gathered kRowsInFlight at a time
constexpr int kRowsInFlight = 8;
constexpr int kEpiWarp0 = 10;
constexpr int kEpiWarps = 8;           // two sets of four (one warp per TMEM lane quarter); set s takes the tiles in accumulator s
constexpr int kMaxStages = 8;
constexpr int kAccBufs = 2;            // accumulators in tensor memory (acc_stride columns each)

struct Args {
  int in_mode;             // 0: uint8 NCHW frames, K order (c, kh, kw), kw == 8;  1: int8 NHWC codes, K order (kh, kw, c)
  int C, H, W, stride, OH, OW, KH, KW;
  int K, Kpad, nkb;        // reduction length, rounded up to 32, 128-byte K blocks
  int N, Npad;             // output channels; N + 1 (the row of ones) rounded up to 16
  int G;                   // samples per work item
  int tiles_item;          // 128-row tiles of a full item
  int sample_bytes;        // input bytes per sample in device memory (a multiple of 16)
  int sample_stride;       // ... and in the staging buffer: mode 0 stages each channel plane with its own copy,
  int plane_bytes;         //     plane_pitch >= plane_bytes apart, the pitch chosen so that the 32 (c, kh) lanes of
  int plane_pitch;         //     a warp hit 32 different banks
  int n_a;                 // operand ring stages
  int acc_stride;          // tensor-memory columns per accumulator: Npad rounded up to a power of two >= 32
  uint32_t ohw_magic, ow_magic;   // ceil(2^32 / (OH*OW)), ceil(2^32 / OW): exact floor divisions of the small row indices
  long long batch, n_items;
  const uint8_t *in;
  const int8_t *img;
  const int *colconst;
  const int *ch_zw;        // per-channel layers: weight zero-points and multipliers per column, else nullptr
  const float *ch_M;
  const LayerParams *params;
  int layer;
  int8_t *out_act;         // [batch][OH][OW][N] int8 codes
  // the last convolution in front of the fully connected tail writes operand blocks for the layer
  // kernel of fc_pair.cu instead (see conv_gemm.cu): sample b = row b, byte pixel * N + channel
  int8_t *blk_out;
  int *blk_rs;
  int blk_nkb, blk_unsigned;
  int *zero_ptr;           // cleared by this launch (row-sum counters a later launch accumulates into), or nullptr
  long long zero_len;
  long long out_elems;     // per sample, for the debug tap's (c, h, w) order
  int *dbg_acc;
  int8_t *dbg_act;
  int *status;
};

struct __align__(16) Barriers {
  uint64_t w_full;           // the weight image has landed
  uint64_t w_ready;          // ... and carries its row of ones
  uint64_t in_full[2], in_empty[2];
  uint64_t a_full[kMaxStages], a_empty[kMaxStages];
  uint64_t acc_full[kAccBufs], acc_empty[kAccBufs];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, const uint4 &v) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void sts64(uint32_t addr, uint32_t lo, uint32_t hi) {
  asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(lo), "r"(hi) : "memory");
}

// kRowsInFlight operand rows of a tile, one warp instruction per row and step; nothing in the loop depends
// on the row.  Rows past the item's last one read whatever the staging buffer holds: their accumulators
// are never used (operand rows are independent of one another).
//   rs       the rows' entries of the row-offset table (kGatherWarps apart)
//   src[st]  shared address of the staged input + the lane's offset inside a receptive field
//   dst[st]  shared address of the lane's bytes in the first of the rows (swizzle folded in); rows kGatherWarps * 128 apart
// kPlanes: uint8 NCHW input, 8 bytes per lane (code = u - 128), else int8 NHWC, 16 bytes per lane.
template <bool kPlanes>
__device__ __forceinline__ void gather_rows(const int *rs, const uint32_t (&src)[2], const uint32_t (&dst)[2],
                                            const bool (&data_ok)[2], const bool (&slot_ok)[2]) {
  constexpr int U = kRowsInFlight;
  constexpr uint32_t kDstStride = (uint32_t)kGatherWarps << 7;
  uint32_t off[U];
#pragma unroll
  for (int u = 0; u < U; ++u) off[u] = (uint32_t)rs[u * kGatherWarps];
#pragma unroll
  for (int st = 0; st < 2; ++st) {
    if (!slot_ok[st]) continue;
    if (kPlanes) {
      uint32_t lo[U], hi[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        lo[u] = 0u; hi[u] = 0u;
        if (data_ok[st]) { lo[u] = lds32(src[st] + off[u]) ^ 0x80808080u; hi[u] = lds32(src[st] + off[u] + 4) ^ 0x80808080u; }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) sts64(dst[st] + (uint32_t)u * kDstStride, lo[u], hi[u]);
    } else {
      uint4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) v[u] = data_ok[st] ? lds128(src[st] + off[u]) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int u = 0; u < U; ++u) sts128(dst[st] + (uint32_t)u * kDstStride, v[u]);
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
conv_staged_kernel(const __grid_constant__ Args A) {
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicMax(A.status, (int)ACTORQ_ERR_CUDA);
    return;
  }
  const int w_bytes = A.nkb * A.Npad * 128;                       // resident weights (a multiple of 2 KB)
  const int in_bytes = (A.G * A.sample_stride + 1023) & ~1023;    // one staging buffer
  uint8_t *a_ring = smem;
  uint8_t *w_res = a_ring + A.n_a * kStageBytes;
  uint8_t *in_s = w_res + ((w_bytes + 1023) & ~1023);
  Barriers *bars = reinterpret_cast<Barriers *>(in_s + 2 * in_bytes);
  int *cc_s = reinterpret_cast<int *>(bars + 1);                  // [128] column constants
  int *row_src = cc_s + kChunkN;                                   // [tiles_item * 128] where a row's receptive field starts
  int *row_pix = row_src + A.tiles_item * kTileM;                  // [tiles_item * 128] (sample in item) << 16 | output pixel
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int *abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    mbar_init(&bars->w_full, 1);
    mbar_init(&bars->w_ready, kEpiWarps);
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->in_full[b], 1); mbar_init(&bars->in_empty[b], kGatherWarps); }
    for (int s = 0; s < kMaxStages; ++s) { mbar_init(&bars->a_full[s], kGatherWarps); mbar_init(&bars->a_empty[s], 1); }
    for (int b = 0; b < kAccBufs; ++b) { mbar_init(&bars->acc_full[b], 1); mbar_init(&bars->acc_empty[b], 4); }
    mbar_init(&bars->drain, 1);
    bars->abort_flag = 0;
    if (blockIdx.x == 0) A.status[7] = (int)smem_u32(bars);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // no more tensor memory than the two accumulators need: giving it back at the end takes time in
  // proportion to the columns held (about 11 us for all 512 on this GPU)
  if (warp == 1) tmem_alloc(&bars->tmem_base, (uint32_t)(kAccBufs * A.acc_stride));
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  // Launched as a programmatic dependent: the set-up above overlaps the tail of the previous kernel
  // on the stream; nothing below (reads of the input, the weight image and the layer constants,
  // writes of the output) runs before that kernel has completed.
  griddep_launch_dependents();
  griddep_wait();
  if (A.zero_ptr != nullptr)
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < A.zero_len; i += (long long)gridDim.x * kThreads)
      A.zero_ptr[i] = 0;

  const int ohw = A.OH * A.OW;
  // per row of an item: the offset of its receptive field's corner inside the staged input, and (sample, pixel)
  for (int ir = threadIdx.x; ir < A.tiles_item * kTileM; ir += kThreads) {
    const int gi = (int)__umulhi((uint32_t)ir, A.ohw_magic);
    const int pix = ir - gi * ohw;
    const int oh = (int)__umulhi((uint32_t)pix, A.ow_magic), ow = pix - oh * A.OW;
    const int sp = (oh * A.stride) * A.W + ow * A.stride;
    row_src[ir] = gi < A.G ? gi * A.sample_stride + (A.in_mode == 1 ? sp * A.C : sp) : 0;
    row_pix[ir] = (gi << 16) | pix;
  }
  if (threadIdx.x < kChunkN) cc_s[threadIdx.x] = threadIdx.x < A.N ? __ldg(A.colconst + threadIdx.x) : 0;
  __syncthreads();
  // items of this CTA: blockIdx.x, + gridDim.x, ...; an item holds n_s <= G samples = n_s * ohw rows
  auto item_samples = [&](long long item) -> int {
    const long long left = A.batch - item * A.G;
    return (int)(left < A.G ? left : A.G);
  };

  if (warp == 0) {
    // ---------------- producer: the weight image once, then one bulk copy per item ----------------
    if (elect_one()) {
      mbar_expect_tx(&bars->w_full, (uint32_t)w_bytes);
      for (int kb = 0; kb < A.nkb; ++kb)
        bulk_g2s(w_res + kb * A.Npad * 128, A.img + ((size_t)kb << 14), (uint32_t)A.Npad * 128, &bars->w_full);
    }
    __syncwarp();
    uint32_t i = 0;
    bool ok = true;
    for (long long item = blockIdx.x; item < A.n_items && ok; item += gridDim.x, ++i) {
      const int buf = i & 1;
      if (i >= 2) {
        ok = mbar_wait_warp(&bars->in_empty[buf], ((i >> 1) - 1) & 1, abort_flag, A.status);
        if (!ok) break;
      }
      if (elect_one()) {
        const int n_s = item_samples(item);
        const uint32_t bytes = (uint32_t)n_s * (uint32_t)A.sample_bytes;
        const uint8_t *src = A.in + (size_t)item * A.G * A.sample_bytes;
        mbar_expect_tx(&bars->in_full[buf], bytes);
        if (A.in_mode == 1 || A.plane_pitch == A.plane_bytes) {
          bulk_g2s(in_s + buf * in_bytes, src, bytes, &bars->in_full[buf]);
        } else {                                           // one copy per channel plane, planes plane_pitch apart
          for (int gi = 0; gi < n_s; ++gi)
            for (int c = 0; c < A.C; ++c)
              bulk_g2s(in_s + buf * in_bytes + gi * A.sample_stride + c * A.plane_pitch,
                       src + (size_t)gi * A.sample_bytes + (size_t)c * A.plane_bytes, (uint32_t)A.plane_bytes, &bars->in_full[buf]);
        }
      }
      __syncwarp();
    }
    if (!ok) for (int k = 0; k < 64; ++k) __nanosleep(1000);     // bulk copies still in flight into this CTA
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    int s = 0;
    uint32_t ph = 0, tc = 0;
    const uint32_t idesc = instr_desc(A.Npad);
    bool ok = mbar_wait_warp(&bars->w_ready, 0, abort_flag, A.status);
    tc_fence_after();
    for (long long item = blockIdx.x; item < A.n_items && ok; item += gridDim.x) {
      const int n_tiles = (item_samples(item) * ohw + kTileM - 1) / kTileM;
      for (int t = 0; t < n_tiles && ok; ++t, ++tc) {
        const uint32_t buf = tc & (kAccBufs - 1), use = tc / kAccBufs;
        ok = mbar_wait_warp(&bars->acc_empty[buf], (use & 1) ^ 1, abort_flag, A.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem + buf * A.acc_stride;
        for (int kb = 0; kb < A.nkb; ++kb) {
          ok = mbar_wait_warp(&bars->a_full[s], ph, abort_flag, A.status);
          if (!ok) break;
          tc_fence_after();
          const int ksteps = min(128, A.Kpad - kb * 128) >> 5;
          const uint32_t a_lo = desc_lo(smem_u32(a_ring + s * kStageBytes));
          const uint32_t b_lo = desc_lo(smem_u32(w_res + kb * A.Npad * 128));
          if (elect_one()) {
            if (ksteps == 4) {
              mma4_i8_ss(d_tmem, a_lo, b_lo, kDescHi, idesc, kb != 0);
            } else {
              const uint64_t adesc = ((uint64_t)kDescHi << 32) | a_lo, bdesc = ((uint64_t)kDescHi << 32) | b_lo;
              for (int ks = 0; ks < ksteps; ++ks)
                mma_i8(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), idesc, (kb | ks) != 0);
            }
            mma_commit(&bars->a_empty[s]);
            if (kb + 1 == A.nkb) mma_commit(&bars->acc_full[buf]);
          }
          __syncwarp();
          if (++s == A.n_a) { s = 0; ph ^= 1; }
        }
      }
    }
    // leaving (done or aborted): none of this thread's MMAs may still run when TMEM is freed below
    if (elect_one()) mma_commit(&bars->drain);
    __syncwarp();
    volatile int never = 0;
    mbar_wait_warp(&bars->drain, 0, &never, A.status);
  } else if (warp < kEpiWarp0) {
    // ---------------- gather (warps 2..9): a warp per output pixel, lanes over the receptive field ----------------
    const int gw = warp - kGatherWarp0;
    // what this lane fetches in each of the (at most two) steps over a row's K bytes:
    //   mode 1: 16-byte piece j = 32 step + lane of the row, K order (kh, kw, c): input offset of its 16 channels
    //   mode 0: 8 bytes q = 32 step + lane = (c, kh): input row segment kw = 0..7 (lane pairs form a 16-byte piece)
    int src_off[2], piece[2];
    uint32_t dst_lane[2];     // the lane's bytes in row gw of a ring stage; its rows, kGatherWarps apart, share row & 7
    bool data_ok[2], slot_ok[2];
    const uint32_t ring_addr = smem_u32(a_ring);
#pragma unroll
    for (int st = 0; st < 2; ++st) {
      const int j = st * 32 + lane;
      if (A.in_mode == 1) {
        const int seg = (A.KW * A.C) >> 4;                 // 16-byte pieces per kh row of the receptive field
        const int kh = j / seg, within = j - kh * seg;
        src_off[st] = kh * A.W * A.C + within * 16;
        piece[st] = j;
        data_ok[st] = j < (A.K >> 4);
        slot_ok[st] = j < (A.Kpad >> 4);
        dst_lane[st] = ((uint32_t)gw << 7) + (((uint32_t)(piece[st] ^ gw) & 7) << 4);
      } else {
        const int c = j / A.KH, kh = j - c * A.KH;
        src_off[st] = c * A.plane_pitch + kh * A.W;
        piece[st] = j >> 1;
        data_ok[st] = j < A.C * A.KH;
        slot_ok[st] = j < (A.Kpad >> 3);                    // every lane stores its 8 bytes (half of a 16-byte piece)
        dst_lane[st] = ((uint32_t)gw << 7) + (((uint32_t)(piece[st] ^ gw) & 7) << 4) + ((uint32_t)(lane & 1) << 3);
      }
    }
    int s = 0;
    uint32_t ph = 0, tc = 0, i = 0;
    bool ok = true;
    for (long long item = blockIdx.x; item < A.n_items && ok; item += gridDim.x, ++i) {
      const int buf = i & 1;
      const int n_tiles = (item_samples(item) * ohw + kTileM - 1) / kTileM;
      ok = mbar_wait_warp(&bars->in_full[buf], (i >> 1) & 1, abort_flag, A.status);
      if (!ok) break;
      const uint32_t in_addr = smem_u32(in_s + buf * in_bytes);
      const uint32_t src[2] = {in_addr + (uint32_t)src_off[0], in_addr + (uint32_t)src_off[1]};
      for (int t = 0; t < n_tiles && ok; ++t, ++tc) {
        // the tile's nkb operand stages: wait until the MMAs that read their previous contents are done
        uint32_t stage_base[2] = {0u, 0u};
        {
          int s2 = s;
          uint32_t ph2 = ph;
          for (int kb = 0; kb < A.nkb; ++kb) {
            ok = mbar_wait_warp(&bars->a_empty[s2], ph2 ^ 1, abort_flag, A.status);
            if (!ok) break;
#pragma unroll
            for (int st = 0; st < 2; ++st)
              if ((piece[st] >> 3) == kb) stage_base[st] = (uint32_t)s2 * kStageBytes;
            if (++s2 == A.n_a) { s2 = 0; ph2 ^= 1; }
          }
          if (!ok) break;
        }
        // the warp's rows, kRowsInFlight at a time so that their loads and stores overlap (one row alone is a
        // chain of shared-memory latencies)
        const uint32_t dst[2] = {ring_addr + stage_base[0] + dst_lane[0], ring_addr + stage_base[1] + dst_lane[1]};
#pragma unroll
        for (int u0 = 0; u0 < kRowsWarp; u0 += kRowsInFlight) {
          const int *rs = row_src + t * kTileM + gw + u0 * kGatherWarps;
          const uint32_t d[2] = {dst[0] + ((uint32_t)(u0 * kGatherWarps) << 7), dst[1] + ((uint32_t)(u0 * kGatherWarps) << 7)};
          if (A.in_mode == 1) gather_rows<false>(rs, src, d, data_ok, slot_ok);
          else gather_rows<true>(rs, src, d, data_ok, slot_ok);
        }
        fence_proxy_async();
        __syncwarp();
        for (int kb = 0; kb < A.nkb; ++kb) {
          if (lane == 0) mbar_arrive(&bars->a_full[s]);
          if (++s == A.n_a) { s = 0; ph ^= 1; }
        }
      }
      __syncwarp();
      if (ok && lane == 0) mbar_arrive(&bars->in_empty[buf]);     // this warp is done with the staged input
    }
  } else {
    // ---------------- epilogue (warps 10..17): two sets, one warp per TMEM lane quarter each ----------------
    const int quarter = warp & 3;
    const uint32_t set = (uint32_t)(warp - kEpiWarp0) >> 2;      // this warp's accumulator: tiles tc with tc % 2 == set
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const LayerParams p = A.params[A.layer];
    const float hi_f = (float)(127 - p.z_out);
    const bool fast = (p.M >= 0x1p-13f) && ((long long)A.K * 65025 + p.bias_absmax < (1ll << 29));
    const int mode = !fast ? 0 : ((p.z_out == -128 && p.M < 0x1p-8f) ? 2 : 1);
    uint32_t tc = 0;
    // the row of ones behind the N weight rows of every K block (all its bytes equal: the swizzle does not matter)
    bool ok = mbar_wait_warp(&bars->w_full, 0, abort_flag, A.status);
    if (ok) {
      const int e = warp - kEpiWarp0;
      for (int i = e * 32 + lane; i < A.nkb * 8; i += kEpiWarps * 32)
        *reinterpret_cast<uint4 *>(w_res + (i >> 3) * A.Npad * 128 + A.N * 128 + (i & 7) * 16) =
            make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->w_ready);
    }
    for (long long item = blockIdx.x; item < A.n_items && ok; item += gridDim.x) {
      const int rows_valid = item_samples(item) * ohw;
      const int n_tiles = (rows_valid + kTileM - 1) / kTileM;
      for (int t = 0; t < n_tiles && ok; ++t, ++tc) {
        const uint32_t buf = tc & (kAccBufs - 1), use = tc / kAccBufs;
        if (buf != set) continue;
        ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_full[buf], use & 1, abort_flag, A.status));
        if (!ok) break;
        tc_fence_after();
        const int ir = t * kTileM + row;
        const bool m_ok = ir < rows_valid;
        const int gp = row_pix[ir];
        const int gi = m_ok ? gp >> 16 : 0;
        const int pix = m_ok ? gp & 0xffff : 0;
        const long long b = item * A.G + gi;
        const long long m = b * ohw + pix;
        // accumulator column N = the row's codes times the weight image's row of ones = their sum
        const int rowsum_a = (int)tmem_ld1_wait(tmem + lane_addr + buf * A.acc_stride + A.N);
        const int rterm = -p.z_w * rowsum_a;
        int blk_sum = 0;
        for (int col0 = 0; col0 < A.N; col0 += 32) {
          uint32_t r[32];
          tmem_ld32_wait(tmem + lane_addr + buf * A.acc_stride + col0, r);
          const int n0 = col0;
          const int4 *cc4 = reinterpret_cast<const int4 *>(cc_s + n0);
          if (A.dbg_acc && m_ok) {
            for (int j = 0; j < 32; ++j)
              if (n0 + j < A.N)
                A.dbg_acc[b * A.out_elems + (long long)(n0 + j) * ohw + pix] =
                    (int)(r[j] + (uint32_t)cc_s[n0 + j] + (uint32_t)(A.ch_zw ? -__ldg(A.ch_zw + n0 + j) * rowsum_a : rterm));
          }
          uint32_t packed[8];
          if (A.ch_zw) requant32_pc(r, A.colconst + n0, A.ch_zw + n0, A.ch_M + n0, rowsum_a, hi_f, p.z_out, packed);
          else if (mode == 2) requant32<2, true>(r, cc4, rterm, p.M, hi_f, p.z_out, packed);
          else if (mode == 1) requant32<1, true>(r, cc4, rterm, p.M, hi_f, p.z_out, packed);
          else requant32<0, true>(r, cc4, rterm, p.M, hi_f, p.z_out, packed);
          if (A.dbg_act && m_ok) {
            for (int j = 0; j < 32; ++j)
              if (n0 + j < A.N)
                A.dbg_act[b * A.out_elems + (long long)(n0 + j) * ohw + pix] = (int8_t)(packed[j >> 2] >> (8 * (j & 3)));
          }
          if (m_ok && A.blk_out != nullptr) {
            if (A.blk_unsigned) {
#pragma unroll
              for (int j = 0; j < 8; ++j) packed[j] ^= 0x80808080u;
            }
            const uint32_t r128 = (uint32_t)(b & 127);
            int8_t *row_blk = A.blk_out + ((((b >> 7) * A.blk_nkb) << 14) + (r128 << 7));
#pragma unroll
            for (int h = 0; h < 2; ++h) {                                    // 16 codes = one 16-byte piece of the row
              if (n0 + 16 * (h + 1) > A.N) break;                            // N is a multiple of 16
              const long long k = (long long)pix * A.N + n0 + 16 * h;        // byte of the tail's input row
              const uint32_t kc = ((uint32_t)k & 127) >> 4;
              *reinterpret_cast<uint4 *>(row_blk + ((k >> 7) << 14) + ((kc ^ (r128 & 7)) << 4)) =
                  make_uint4(packed[4 * h], packed[4 * h + 1], packed[4 * h + 2], packed[4 * h + 3]);
#pragma unroll
              for (int j = 4 * h; j < 4 * h + 4; ++j)
                blk_sum = A.blk_unsigned ? (int)__dp4a(packed[j], 0x01010101u, (unsigned)blk_sum) : __dp4a((int)packed[j], 0x01010101, blk_sum);
            }
          } else if (m_ok) {
            int8_t *o = A.out_act + m * A.N + n0;
            if (n0 + 16 <= A.N) *reinterpret_cast<uint4 *>(o) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            if (n0 + 32 <= A.N) *reinterpret_cast<uint4 *>(o + 16) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
          }
        }
        if (A.blk_out != nullptr && m_ok) atomicAdd(A.blk_rs + b, blk_sum);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->acc_empty[buf]);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, (uint32_t)(kAccBufs * A.acc_stride));
  }
}

}  // namespace cst

// ---- host side ------------------------------------------------------------------------------

static int cst_round_up(int v, int m) { return (v + m - 1) / m * m; }

struct CstPlan { bool ok; int G, n_a, tiles_item, smem_bytes, sample_bytes, sample_stride, plane_bytes, plane_pitch, in_mode; };

// Does the staged kernel take convolution layer l of this (tensor-core conv path) policy, and with
// which samples-per-item and ring depth?  G minimises (rounds of items over the SMs) x (tiles per item).
static CstPlan plan_conv_staged(const actorq_policy *p, int l, long long batch) {
  CstPlan pl = {false, 0, 0, 0, 0, 0, 0, 0, 0, 0};
  const LayerGeom &g = p->layers[l].g;
  if (g.kind != ACTORQ_CONV2D || g.N > 112 || (g.N & 15)) return pl;       // N + 1 columns (the row sums) fit one accumulator
  pl.in_mode = (l == 0) ? 0 : 1;
  if (pl.in_mode == 0) {
    if (p->obs_dtype != ACTORQ_OBS_U8_DIV255 || g.kw != 8 || (g.stride & 3) || (g.in_w & 3) || g.K > 512) return pl;
    pl.sample_bytes = g.in_c * g.in_h * g.in_w;
    pl.plane_bytes = g.in_h * g.in_w;
    pl.plane_pitch = pl.plane_bytes;
    if ((pl.plane_bytes & 15) == 0) {
      // the pitch (plane + 0, 16, .. 112 bytes) for which the banks of the lanes' words, lane = (c, kh) at
      // byte c * pitch + kh * in_w, collide least
      int best = 1 << 30;
      for (int pad = 0; pad < 128; pad += 16) {
        int hits[32] = {0}, worst = 0;
        for (int q = 0; q < 32 && q < g.in_c * g.kh; ++q) {
          const int c = q / g.kh, kh = q - c * g.kh;
          const int bank = ((c * (pl.plane_bytes + pad) + kh * g.in_w) >> 2) & 31;
          if (++hits[bank] > worst) worst = hits[bank];
        }
        if (worst < best) { best = worst; pl.plane_pitch = pl.plane_bytes + pad; }
      }
    }
    pl.sample_stride = g.in_c * pl.plane_pitch;
  } else {
    if ((g.in_c & 15) || g.K > 1024) return pl;
    pl.sample_bytes = g.in_h * g.in_w * g.in_c;
    pl.sample_stride = pl.sample_bytes;
  }
  if (pl.sample_bytes & 15) return pl;
  const int nkb = (g.K + 127) / 128;
  const int ohw = g.out_h * g.out_w;
  const int w_bytes = cst_round_up(nkb * cst_round_up(g.N + 1, 16) * 128, 1024);
  const int fixed = w_bytes + (int)sizeof(cst::Barriers) + kChunkN * (int)sizeof(int) + 1024;
  long long best_cost = -1;
  for (int G = 1; G <= 16; ++G) {
    if ((long long)G * ohw > 65535) break;
    const int in_bytes = cst_round_up(G * pl.sample_stride, 1024);
    const int tiles = (G * ohw + kTileM - 1) / kTileM;
    if (tiles > 16) break;
    const int table_bytes = 2 * tiles * kTileM * (int)sizeof(int);
    int n_a = (kMaxSmem - fixed - 2 * in_bytes - table_bytes) / kStageBytes;
    if (n_a > cst::kMaxStages) n_a = cst::kMaxStages;
    if (n_a < nkb) break;                                  // a tile's K blocks must fit the ring (larger G: less room still)
    const long long items = (batch + G - 1) / G;
    const long long rounds = (items + p->sm_count - 1) / p->sm_count;
    const long long cost = rounds * tiles * 16 + (n_a < 2 * nkb ? 1 : 0);      // ties: the deeper ring
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      pl.G = G; pl.n_a = n_a; pl.tiles_item = tiles;
      pl.smem_bytes = n_a * kStageBytes + w_bytes + 2 * in_bytes + (int)sizeof(cst::Barriers) + kChunkN * (int)sizeof(int) + table_bytes;
    }
  }
  pl.ok = best_cost >= 0;
  return pl;
}

bool conv_staged_supported(const actorq_policy *p, int l, long long batch) { return plan_conv_staged(p, l, batch).ok; }

// Launches convolution layer l on the staged kernel.  in: the layer's input (the caller's frames or the
// previous layer's NHWC codes); out_act / blk_*: where the codes go (see cst::Args).
int launch_conv_staged(actorq_policy *p, int l, const void *in, long long batch, int8_t *out_act,
                       int8_t *blk_out, int *blk_rs, int blk_nkb, int blk_unsigned, int *zero_ptr, long long zero_len,
                       int *dbg_acc, int8_t *dbg_act, cudaStream_t st) {
  const CstPlan pl = plan_conv_staged(p, l, batch);
  if (!pl.ok) return ACTORQ_ERR_UNSUPPORTED;
  static bool attr_set[64] = {false};
  if (p->device >= 0 && p->device < 64 && !attr_set[p->device]) {
    if (cudaFuncSetAttribute(cst::conv_staged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
      return ACTORQ_ERR_CUDA;
    attr_set[p->device] = true;
  }
  const LayerDev &L = p->layers[l];
  const LayerGeom &g = L.g;
  cst::Args A;
  memset(&A, 0, sizeof(A));
  A.in_mode = pl.in_mode;
  A.C = g.in_c; A.H = g.in_h; A.W = g.in_w; A.stride = g.stride; A.OH = g.out_h; A.OW = g.out_w; A.KH = g.kh; A.KW = g.kw;
  A.K = g.K; A.Kpad = cst_round_up(g.K, 32); A.nkb = (g.K + 127) / 128;
  A.N = g.N; A.Npad = cst_round_up(g.N + 1, 16);
  A.acc_stride = 32;
  while (A.acc_stride < A.Npad) A.acc_stride *= 2;
  A.G = pl.G; A.tiles_item = pl.tiles_item; A.sample_bytes = pl.sample_bytes; A.n_a = pl.n_a;
  A.sample_stride = pl.sample_stride; A.plane_bytes = pl.plane_bytes; A.plane_pitch = pl.plane_pitch;
  const unsigned long long ohw = (unsigned long long)g.out_h * g.out_w;
  A.ohw_magic = (uint32_t)((0x100000000ull + ohw - 1) / ohw);
  A.ow_magic = (uint32_t)((0x100000000ull + (unsigned long long)g.out_w - 1) / (unsigned long long)g.out_w);
  A.batch = batch;
  A.n_items = (batch + pl.G - 1) / pl.G;
  A.in = (const uint8_t *)in;
  A.img = L.wq_img;
  A.colconst = L.colconst;
  if (g.per_channel) { A.ch_zw = L.ch_zw; A.ch_M = L.ch_M; }
  A.params = p->d_params;
  A.layer = l;
  A.out_act = out_act;
  A.blk_out = blk_out; A.blk_rs = blk_rs; A.blk_nkb = blk_nkb; A.blk_unsigned = blk_unsigned;
  A.zero_ptr = zero_ptr; A.zero_len = zero_len;
  A.out_elems = g.out_elems;
  A.dbg_acc = dbg_acc;
  A.dbg_act = dbg_act;
  A.status = p->d_status;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3((unsigned)(A.n_items < p->sm_count ? A.n_items : p->sm_count));
  cfg.blockDim = dim3(cst::kThreads);
  cfg.dynamicSmemBytes = (size_t)pl.smem_bytes;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, cst::conv_staged_kernel, A) != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_CUDA; }
  p->launches++;
  return ACTORQ_OK;
}

}  // namespace actorq
