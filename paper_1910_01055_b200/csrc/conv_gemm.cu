// Implicit-GEMM int8 convolution / fully connected layer on the tcgen05 tensor cores, one launch
// per layer, for DQN-style policies (paper Section 3.2: the three-layer convolutional Atari policy;
// arithmetic as everywhere: int8 x int8 -> int32, requantize with one binary32 multiply, Eq. 3 head).
//
//   raw[m][n] = sum_k A[m][k] * W[n][k],   m = (sample, oh, ow),  n = output channel,
//                                          k = position inside the receptive field
// Intermediate activations are int8 NHWC in device scratch, so for every layer but the first a
// 16-byte piece of K is 16 consecutive channels of one input pixel: K is ordered (kh, kw, c) and the
// quantizer writes the weight image in that order.  The first layer reads the caller's uint8 NCHW
// frames directly (code = u - 128) with K in the caller's (c, kh, kw) order, 4 bytes at a time.
// A fully connected layer is the same thing with a 1x1 output (its "kernel" covers its whole
// input), so conv1..conv3, FC and the Q-value head all run through this kernel.
//
// One CTA per SM, persistent over work items (128-row tile x group of up to four 128-column
// chunks).  Warps: 0 streams weight tiles (bulk copies, ring), 1 issues the MMAs, 2-9 gather the A
// operand (one lane per output row and half of a 128-byte K block: global loads -> 16-byte swizzled
// shared-memory stores, row sums by dp4a; the gather is latency-bound, so eight warps with two steps
// of loads in flight each), 10-13 drain the accumulators from TMEM, requantize and store.  All
// waits are bounded.
#include "tcgen05.cuh"

namespace actorq {

constexpr int kCgThreads = 448;
constexpr int kCgLoaderWarp0 = 2;
constexpr int kCgLoaderWarps = 8;      // two groups of four: group g gathers 16-byte pieces 4g .. 4g+3 of every K block
constexpr int kCgEpiWarp0 = 10;
constexpr int kCgEpiWarps = 4;
constexpr int kCgMaxStages = 6;
constexpr int kCgRowsumSlots = 16;     // row-sum ring: the loader may run this many items ahead

struct ConvGemmArgs {
  int in_mode;            // 0: uint8 NCHW frames, K order (c, kh, kw);  1: int8 NHWC, K order (kh, kw, c)
  int C, H, W, stride, OH, OW;
  int K, Kpad, nkb;       // reduction length, rounded up to 32, number of 128-byte K blocks
  int N, Npad, nchunk;    // outputs, rounded up to 16, number of 128-column chunks
  int cpg, n_groups;      // chunks per work item, groups per row tile
  int acc_bufs;           // accumulator sets in TMEM (2 when a set is at most 256 columns)
  int n_a, n_b;           // ring depths
  long long M;            // batch * OH * OW
  long long n_items;
  const void *in;
  const int *koff;        // per 16 bytes (mode 1) / 4 bytes (mode 0) of K: offset inside the receptive field
  int n_koff;             // entries of koff
  const int8_t *img;
  const int *colconst;
  const int *ch_zw;       // per-channel layers: [N padded to 128] weight zero-points, multipliers, accumulator
  const float *ch_M;      // units (Section 3.2, per-channel quantization); all nullptr for a per-tensor layer
  const float *ch_P;
  const LayerParams *params;
  int layer, last, head;
  int8_t *out_act;        // [M][N] int8 NHWC (hidden layers)
  // The last convolution in front of the fully connected tail writes its codes where the layer
  // kernel of fc_pair.cu reads them instead: sample b is row b of the tail's input, its (pixel,
  // channel) codes bytes pixel * N + channel of that row, stored as operand blocks (16 KB per 128
  // rows and 128 bytes of the row, 128-byte swizzle), unsigned (code + 128) when blk_unsigned; the
  // sums of a sample's stored codes are added to blk_rs[b].  nullptr for every other layer.
  int8_t *blk_out;
  int *blk_rs;
  int blk_nkb, blk_unsigned;
  float *out;             // [M][N] float (last layer)
  int *actions;
  long long out_elems;    // per sample, for the debug tap's (c, h, w) order
  int *dbg_acc;
  int8_t *dbg_act;
  int *status;
};

struct __align__(16) ConvGemmBarriers {
  uint64_t a_full[kCgMaxStages], a_empty[kCgMaxStages];
  uint64_t b_full[kCgMaxStages], b_empty[kCgMaxStages];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t drain;                 // all MMAs of the issuer have completed (awaited before TMEM is freed)
  uint32_t tmem_base;
  int abort_flag;
  int rowsum[kCgRowsumSlots][2][kTileM];   // per gather group: the sum over its half of every K block
};

__global__ void __launch_bounds__(kCgThreads, 1)
conv_gemm_kernel(const __grid_constant__ ConvGemmArgs A) {
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicMax(A.status, (int)ACTORQ_ERR_CUDA);
    return;
  }
  uint8_t *a_ring = smem;
  uint8_t *b_ring = a_ring + A.n_a * kStageBytes;
  ConvGemmBarriers *bars = reinterpret_cast<ConvGemmBarriers *>(b_ring + A.n_b * kStageBytes);
  // the receptive-field offset table, copied to shared memory once: every gather address depends on
  // an entry, and a global (even cached) lookup in front of each load doubles the load's latency
  int *koff_s = reinterpret_cast<int *>(bars + 1);
  for (int i = threadIdx.x; i < A.n_koff; i += kCgThreads) koff_s[i] = __ldg(A.koff + i);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int *abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kCgMaxStages; ++s) {
      mbar_init(&bars->a_full[s], kCgLoaderWarps); mbar_init(&bars->a_empty[s], 1);
      mbar_init(&bars->b_full[s], 1); mbar_init(&bars->b_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->acc_full[b], 1); mbar_init(&bars->acc_empty[b], kCgEpiWarps); }
    mbar_init(&bars->drain, 1);
    bars->abort_flag = 0;
    if (blockIdx.x == 0) A.status[7] = (int)smem_u32(bars);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&bars->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  const int acc_cols = A.cpg * kChunkN;
  // Everything above is set-up that reads nothing an earlier kernel of the stream writes; from here
  // on the layer's input, the weight image and the layer constants are read.
  griddep_launch_dependents();
  griddep_wait();

  if (warp == 0) {
    // ---------------- weight-tile producer ----------------
    int s = 0; uint32_t ph = 0; bool ok = true;
    for (long long item = blockIdx.x; item < A.n_items && ok; item += gridDim.x) {
      const int g = (int)(item % A.n_groups);
      for (int kb = 0; kb < A.nkb && ok; ++kb) {
        for (int ci = 0; ci < A.cpg; ++ci) {
          const int c = g * A.cpg + ci;
          if (c >= A.nchunk) break;
          const uint32_t bytes = (uint32_t)min(kChunkN, A.Npad - c * kChunkN) * 128;
          ok = mbar_wait_warp(&bars->b_empty[s], ph ^ 1, abort_flag, A.status);
          if (!ok) break;
          if (elect_one()) {
            mbar_expect_tx(&bars->b_full[s], bytes);
            bulk_g2s(b_ring + s * kStageBytes, A.img + ((size_t)(c * A.nkb + kb) << 14), bytes, &bars->b_full[s]);
          }
          __syncwarp();
          if (++s == A.n_b) { s = 0; ph ^= 1; }
        }
      }
    }
    if (!ok) for (int i = 0; i < 64; ++i) __nanosleep(1000);
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    int sa = 0, sb = 0; uint32_t pha = 0, phb = 0, it = 0; bool ok = true;
    for (long long item = blockIdx.x; item < A.n_items && ok; item += gridDim.x, ++it) {
      const int g = (int)(item % A.n_groups);
      const int buf = A.acc_bufs == 2 ? (it & 1) : 0;
      const uint32_t use = A.acc_bufs == 2 ? (it >> 1) : it;
      ok = mbar_wait_warp(&bars->acc_empty[buf], (use & 1) ^ 1, abort_flag, A.status);
      if (!ok) break;
      tc_fence_after();
      for (int kb = 0; kb < A.nkb && ok; ++kb) {
        ok = mbar_wait_warp(&bars->a_full[sa], pha, abort_flag, A.status);
        if (!ok) break;
        tc_fence_after();
        const int ksteps = min(128, A.Kpad - kb * 128) >> 5;
        const uint64_t adesc = smem_desc(smem_u32(a_ring + sa * kStageBytes));
        const bool last_kb = (kb + 1 == A.nkb);
        for (int ci = 0; ci < A.cpg; ++ci) {
          const int c = g * A.cpg + ci;
          if (c >= A.nchunk) break;
          const uint32_t idesc = instr_desc(min(kChunkN, A.Npad - c * kChunkN));
          ok = mbar_wait_warp(&bars->b_full[sb], phb, abort_flag, A.status);
          if (!ok) break;
          tc_fence_after();
          const uint64_t bdesc = smem_desc(smem_u32(b_ring + sb * kStageBytes));
          const uint32_t d_tmem = tmem + buf * acc_cols + ci * kChunkN;
          const bool last_c = (ci + 1 == A.cpg) || (c + 1 == A.nchunk);
          if (elect_one()) {
            if (ksteps == 4) {     // a whole K block: four MMAs in one statement
              mma4_i8_ss(d_tmem, desc_lo(smem_u32(a_ring + sa * kStageBytes)), desc_lo(smem_u32(b_ring + sb * kStageBytes)),
                         kDescHi, idesc, kb != 0);
            } else {
              for (int ks = 0; ks < ksteps; ++ks)
                mma_i8(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), idesc, (kb | ks) != 0);
            }
            mma_commit(&bars->b_empty[sb]);
            if (last_c) {
              mma_commit(&bars->a_empty[sa]);
              if (last_kb) mma_commit(&bars->acc_full[buf]);
            }
          }
          __syncwarp();
          if (++sb == A.n_b) { sb = 0; phb ^= 1; }
        }
        if (++sa == A.n_a) { sa = 0; pha ^= 1; }
      }
    }
    // Leaving (done or aborted): none of this thread's MMAs may still run when TMEM is freed below.
    if (elect_one()) mma_commit(&bars->drain);
    __syncwarp();
    volatile int never = 0;                      // this wait must not be cut short by the abort flag
    mbar_wait_warp(&bars->drain, 0, &never, A.status);
  } else if (warp < kCgEpiWarp0) {
    // ---------------- A-operand gather (warps 2..9): one lane per output row and half of a K block ----------------
    // The K blocks of all of this CTA's work items form one stream; the global loads of the next
    // block of the stream (of the next item, at an item's end) are issued before the current one is
    // converted and stored, so a gather warp never sits out a whole memory round trip.
    const int lw = warp - kCgLoaderWarp0;
    const int grp = lw >> 2;                 // which half (64 bytes) of each K block
    const int row = (lw & 3) * 32 + lane;
    const int ohw = A.OH * A.OW;
    struct Step { long long item; int kb; uint32_t it; const uint8_t *src; bool m_ok; };
    auto locate = [&](Step &t) {          // row decode of the step's work item
      const long long tile = t.item / A.n_groups;
      const long long m = tile * kTileM + row;
      t.m_ok = m < A.M;
      const long long mm = t.m_ok ? m : A.M - 1;
      const long long b = mm / ohw;
      const int pix = (int)(mm - b * ohw);
      const int oh = pix / A.OW, ow = pix - oh * A.OW;
      // origin of the receptive field inside the sample (element offset)
      if (A.in_mode == 0) t.src = (const uint8_t *)A.in + b * (long long)A.C * A.H * A.W + (long long)(oh * A.stride) * A.W + ow * A.stride;
      else t.src = (const uint8_t *)A.in + (b * A.H * A.W + (long long)(oh * A.stride) * A.W + ow * A.stride) * A.C;
    };
    auto advance = [&](Step &t) -> bool { // next step of the stream; false past the end
      if (++t.kb < A.nkb) return true;
      t.kb = 0; t.item += gridDim.x; ++t.it;
      if (t.item >= A.n_items) return false;
      locate(t);
      return true;
    };
    auto issue = [&](const Step &t, uint32_t (&v)[16]) {
      // a K block that lies wholly inside K (all but a layer's last one, usually that too): offsets four
      // at a time from the table, no clamping
      const bool whole = t.kb * 128 + 128 <= A.K;
      if (whole && A.in_mode == 1) {
        const int4 o = *reinterpret_cast<const int4 *>(koff_s + t.kb * 8 + grp * 4);
        const int off[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint4 q = __ldg(reinterpret_cast<const uint4 *>(t.src + off[j]));
          v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
        }
      } else if (whole) {
#pragma unroll
        for (int j4 = 0; j4 < 4; ++j4) {
          const int4 o = *reinterpret_cast<const int4 *>(koff_s + t.kb * 32 + grp * 16 + j4 * 4);
          v[4 * j4 + 0] = __ldg(reinterpret_cast<const uint32_t *>(t.src + o.x));
          v[4 * j4 + 1] = __ldg(reinterpret_cast<const uint32_t *>(t.src + o.y));
          v[4 * j4 + 2] = __ldg(reinterpret_cast<const uint32_t *>(t.src + o.z));
          v[4 * j4 + 3] = __ldg(reinterpret_cast<const uint32_t *>(t.src + o.w));
        }
      } else if (A.in_mode == 1) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int k = t.kb * 128 + grp * 64 + j * 16;
          const int kk = k < A.K ? k : 0;                        // clamped address, masked value
          const uint4 q = __ldg(reinterpret_cast<const uint4 *>(t.src + koff_s[kk >> 4]));
          v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int k = t.kb * 128 + grp * 64 + j * 4;
          const int kk = k < A.K ? k : 0;
          v[j] = __ldg(reinterpret_cast<const uint32_t *>(t.src + koff_s[kk >> 2]));
        }
      }
    };
    int sa = 0; uint32_t pha = 0; int rsum = 0;
    auto finish = [&](const Step &t, uint32_t (&v)[16]) -> bool {
      if (!mbar_wait_warp(&bars->a_empty[sa], pha ^ 1, abort_flag, A.status)) return false;
      uint8_t *dst = a_ring + sa * kStageBytes + ((uint32_t)row << 7);
      if (t.kb == 0) rsum = 0;
      if (t.m_ok && t.kb * 128 + 128 <= A.K) {                   // nothing to mask
        const uint32_t flip = (A.in_mode == 0) ? 0x80808080u : 0u;   // code = u - 128
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          v[j] ^= flip;
          rsum = __dp4a((int)v[j], 0x01010101, rsum);
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int k = t.kb * 128 + grp * 64 + j * 4;
          uint32_t w = v[j];
          if (A.in_mode == 0) w ^= 0x80808080u;                    // code = u - 128
          if (!t.m_ok || k >= A.K) w = 0u;                         // rows / K outside: code 0
          v[j] = w;
          rsum = __dp4a((int)w, 0x01010101, rsum);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<uint4 *>(dst + (((uint32_t)(grp * 4 + j) ^ ((uint32_t)row & 7)) << 4)) =
            make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
      if (t.kb + 1 == A.nkb) bars->rowsum[t.it % kCgRowsumSlots][grp][row] = rsum;
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->a_full[sa]);
      if (++sa == A.n_a) { sa = 0; pha ^= 1; }
      return true;
    };
    uint32_t va[16], vb[16];
    Step cur = {(long long)blockIdx.x, 0, 0u, nullptr, false};
    bool more = cur.item < A.n_items, ok = true;
    if (more) { locate(cur); issue(cur, va); }
    while (more && ok) {
      Step nxt = cur;
      const bool has_b = advance(nxt);
      if (has_b) issue(nxt, vb);
      ok = finish(cur, va);
      if (!ok || !has_b) break;
      cur = nxt;
      more = advance(cur);
      if (more) issue(cur, va);
      ok = finish(nxt, vb);
    }
  } else {
    // ---------------- epilogue (warps 10..13): one warp per TMEM lane quarter ----------------
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const LayerParams p = A.params[A.layer];
    const float hi_f = (float)(127 - p.z_out);
    const bool fast = (p.M >= 0x1p-13f) && ((long long)A.K * 65025 + p.bias_absmax < (1ll << 29));
    const int mode = !fast ? 0 : ((p.z_out == -128 && p.M < 0x1p-8f) ? 2 : 1);
    const int ohw = A.OH * A.OW;
    uint32_t it = 0; bool ok = true;
    for (long long item = blockIdx.x; item < A.n_items && ok; item += gridDim.x, ++it) {
      const long long tile = item / A.n_groups;
      const int g = (int)(item % A.n_groups);
      const long long m = tile * kTileM + row;
      const bool m_ok = m < A.M;
      const int buf = A.acc_bufs == 2 ? (it & 1) : 0;
      const uint32_t use = A.acc_bufs == 2 ? (it >> 1) : it;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_full[buf], use & 1, abort_flag, A.status));
      if (!ok) break;
      tc_fence_after();
      // The gather warps stored the row sums before they released the last K block of this item to
      // the MMA issuer, and this accumulator was computed from it.
      const int rowsum_a = bars->rowsum[it % kCgRowsumSlots][0][row] + bars->rowsum[it % kCgRowsumSlots][1][row];
      const int rterm = -p.z_w * rowsum_a;
      const long long b = m_ok ? m / ohw : 0;
      const int pix = m_ok ? (int)(m - b * ohw) : 0;
      float best_v = 0.0f; int best_n = -1;
      int blk_sum = 0;
      for (int ci = 0; ci < A.cpg; ++ci) {
        const int c = g * A.cpg + ci;
        if (c >= A.nchunk) break;
        const int rows_c = min(kChunkN, A.Npad - c * kChunkN);
        for (int col0 = 0; col0 < rows_c; col0 += 32) {
          uint32_t r[32];
          tmem_ld32_wait(tmem + lane_addr + buf * acc_cols + ci * kChunkN + col0, r);
          const int n0 = c * kChunkN + col0;
          const int4 *cc4 = reinterpret_cast<const int4 *>(A.colconst + n0);
          if (A.dbg_acc && m_ok) {
            for (int j = 0; j < 32; ++j)
              if (n0 + j < A.N)
                A.dbg_acc[b * A.out_elems + (long long)(n0 + j) * ohw + pix] =
                    (int)(r[j] + (uint32_t)__ldg(A.colconst + n0 + j) + (uint32_t)(A.ch_zw ? -__ldg(A.ch_zw + n0 + j) * rowsum_a : rterm));
          }
          if (!A.last) {
            uint32_t packed[8];
            if (A.ch_zw) requant32_pc(r, A.colconst + n0, A.ch_zw + n0, A.ch_M + n0, rowsum_a, hi_f, p.z_out, packed);
            else if (mode == 2) requant32<2>(r, cc4, rterm, p.M, hi_f, p.z_out, packed);
            else if (mode == 1) requant32<1>(r, cc4, rterm, p.M, hi_f, p.z_out, packed);
            else requant32<0>(r, cc4, rterm, p.M, hi_f, p.z_out, packed);
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
                if (n0 + 16 * (h + 1) > A.N) break;                            // N is a multiple of 16 on this path
                const long long k = (long long)pix * A.N + n0 + 16 * h;        // byte of the tail's input row
                const uint32_t kc = ((uint32_t)k & 127) >> 4;
                *reinterpret_cast<uint4 *>(row_blk + ((k >> 7) << 14) + ((kc ^ (r128 & 7)) << 4)) =
                    make_uint4(packed[4 * h], packed[4 * h + 1], packed[4 * h + 2], packed[4 * h + 3]);
#pragma unroll
                for (int j = 4 * h; j < 4 * h + 4; ++j)
                  blk_sum = A.blk_unsigned ? (int)__dp4a(packed[j], 0x01010101u, (unsigned)blk_sum) : __dp4a((int)packed[j], 0x01010101, blk_sum);
              }
            } else if (m_ok) {                            // N is a multiple of 16 on this path
              int8_t *o = A.out_act + m * A.N + n0;
              if (n0 + 16 <= A.N) *reinterpret_cast<uint4 *>(o) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
              if (n0 + 32 <= A.N) *reinterpret_cast<uint4 *>(o + 16) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
            }
          } else {
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4) {
              const int4 cc = __ldg(cc4 + j4);
              const int ccv[4] = {cc.x, cc.y, cc.z, cc.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int n = n0 + 4 * j4 + e;
                if (n < A.N) {
                  const int acc = (int)(r[4 * j4 + e] + (uint32_t)ccv[e] + (uint32_t)(A.ch_zw ? -__ldg(A.ch_zw + n) * rowsum_a : rterm));
                  float y = __fmul_rn(__int2float_rn(acc), A.ch_P ? __ldg(A.ch_P + n) : p.P);          // Eq. 3 on the accumulator
                  if (y > best_v || best_n < 0) { best_v = y; best_n = n; }
                  if (A.head == ACTORQ_HEAD_TANH) y = tanhf(y);
                  if (m_ok) A.out[m * A.N + n] = y;
                }
              }
            }
          }
        }
      }
      if (A.last && A.head == ACTORQ_HEAD_ARGMAX && m_ok) A.actions[m] = best_n;
      if (A.blk_out != nullptr && m_ok) atomicAdd(A.blk_rs + b, blk_sum);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->acc_empty[buf]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ---- host side ------------------------------------------------------------------------------

static int cg_round_up(int v, int m) { return (v + m - 1) / m * m; }

// Policies this path takes: uint8 NCHW frames into a convolution whose rows can be read 4 bytes at a
// time; later layers read int8 NHWC with a multiple of 16 channels (an FC layer counts (c, h, w) ->
// (h, w, c) when it follows a convolution, its whole input as channels when it follows an FC layer).
bool conv_gemm_supported(const actorq_policy *p) {
  if (p->obs_dtype != ACTORQ_OBS_U8_DIV255 || p->n_layers < 2) return false;
  const LayerGeom &g0 = p->layers[0].g;
  if (g0.kind != ACTORQ_CONV2D) return false;
  if ((g0.kw & 3) || (g0.stride & 3) || (g0.in_w & 3)) return false;
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerGeom &g = p->layers[l].g;
    const bool last = (l + 1 == p->n_layers);
    if (last ? g.N > 128 : (g.N > 512 || (g.N & 15))) return false;
    if (l > 0) {
      const LayerGeom &gp = p->layers[l - 1].g;
      const int c_in = (g.kind == ACTORQ_CONV2D) ? g.in_c : (gp.kind == ACTORQ_CONV2D ? gp.out_c : g.K);
      if (c_in & 15) return false;
      if (g.kind == ACTORQ_CONV2D && gp.kind != ACTORQ_CONV2D) return false;
    }
  }
  return true;
}

// K permutation the quantizer applies when it writes layer l's weight image on this path:
// canonical (c, kh, kw) -> (kh, kw, c).  Returns false for layers that keep the caller's order.
bool conv_gemm_image_perm(const actorq_policy *p, int l, int *C, int *KH, int *KW) {
  if (!p->conv_ok || l == 0) return false;
  const LayerGeom &g = p->layers[l].g;
  if (g.kind == ACTORQ_CONV2D) { *C = g.in_c; *KH = g.kh; *KW = g.kw; return true; }
  const LayerGeom &gp = p->layers[l - 1].g;
  if (gp.kind == ACTORQ_CONV2D) { *C = gp.out_c; *KH = gp.out_h; *KW = gp.out_w; return true; }
  return false;
}

// per-layer table of receptive-field offsets, one entry per 16 (NHWC) or 4 (NCHW) bytes of K
int conv_gemm_koff_entries(const actorq_policy *p, int l) {
  const LayerGeom &g = p->layers[l].g;
  return (l == 0 && p->obs_dtype == ACTORQ_OBS_U8_DIV255) ? (g.K + 3) / 4 : (g.K + 15) / 16;
}

void conv_gemm_fill_koff(const actorq_policy *p, int l, int *koff) {
  const LayerGeom &g = p->layers[l].g;
  if (l == 0 && p->obs_dtype == ACTORQ_OBS_U8_DIV255) {   // NCHW bytes, K order (c, kh, kw)
    for (int k = 0; k < g.K; k += 4) {
      const int c = k / (g.kh * g.kw), kh = (k / g.kw) % g.kh, kw = k % g.kw;
      koff[k >> 2] = (c * g.in_h + kh) * g.in_w + kw;
    }
    return;
  }
  int C, KW, W;
  if (g.kind == ACTORQ_CONV2D) { C = g.in_c; KW = g.kw; W = g.in_w; }
  else if (l > 0 && p->layers[l - 1].g.kind == ACTORQ_CONV2D) { const LayerGeom &gp = p->layers[l - 1].g; C = gp.out_c; KW = gp.out_w; W = gp.out_w; }
  else { C = g.K; KW = 1; W = 1; }
  for (int k = 0; k < g.K; k += 16) {               // NHWC bytes, K order (kh, kw, c)
    const int c0 = k % C, kw = (k / C) % KW, kh = k / (C * KW);
    koff[k >> 4] = (kh * W + kw) * C + c0;
  }
}

int launch_forward_conv_gemm(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                             int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st) {
  static bool attr_set[64] = {false};
  if (p->device < 64 && !attr_set[p->device]) {
    if (cudaFuncSetAttribute(conv_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
      return ACTORQ_ERR_CUDA;
    attr_set[p->device] = true;
  }
  const void *cur = obs;
  int8_t *bufs[2] = {p->scratch[0], p->scratch[1]};
  // The fully connected layers behind the last convolution run on the CTA-pair layer kernel
  // (fc_pair.cu), fed directly by that convolution's epilogue; where it cannot take them (or no
  // pair of CTAs can be scheduled) they run here like every other layer.
  int l_tail = p->n_layers;
  int8_t *blk = nullptr;
  int *blk_rs = nullptr;
  int blk_nkb = 0;
  int *rs_all = nullptr;          // the tail's row-sum counters: cleared by the kernel of layer l_tail - 2 when that is a
  long long rs_all_len = 0;       // staged convolution (no memset between the kernels of consecutive forwards)
  bool clear_in_kernel = false;
  {
    int lc = -1;
    for (int l = 0; l < p->n_layers; ++l)
      if (p->layers[l].g.kind == ACTORQ_CONV2D) lc = l;
    clear_in_kernel = lc >= 1 && conv_staged_supported(p, lc - 1, batch);
    if (lc >= 0 && lc + 1 < p->n_layers &&
        fc_tail_begin(p, lc + 1, batch, st, &blk, &blk_nkb, &blk_rs, clear_in_kernel ? 0 : 1, &rs_all, &rs_all_len) == ACTORQ_OK)
      l_tail = lc + 1;
  }
  for (int l = 0; l < l_tail; ++l) {
    const LayerDev &L = p->layers[l];
    const LayerGeom &g = L.g;
    const bool last = (l + 1 == p->n_layers);
    if (conv_staged_supported(p, l, batch)) {      // convolutions: input staged in shared memory
      const bool feeds_tail = (l + 1 == l_tail && l_tail < p->n_layers);
      const bool clears = clear_in_kernel && l_tail < p->n_layers && l == l_tail - 2;
      const int rc = launch_conv_staged(p, l, cur, batch, feeds_tail ? nullptr : bufs[l & 1], feeds_tail ? blk : nullptr,
                                        feeds_tail ? blk_rs : nullptr, blk_nkb, (feeds_tail && p->act[l_tail].z == -128) ? 1 : 0,
                                        clears ? rs_all : nullptr, clears ? rs_all_len : 0,
                                        (l == dbg_layer) ? dbg_acc : nullptr, (l == dbg_layer) ? dbg_act : nullptr, st);
      if (rc != ACTORQ_OK) return rc;
      cur = bufs[l & 1];
      continue;
    }
    ConvGemmArgs A;
    memset(&A, 0, sizeof(A));
    A.in_mode = (l == 0) ? 0 : 1;
    if (g.kind == ACTORQ_CONV2D) {
      A.C = g.in_c; A.H = g.in_h; A.W = g.in_w; A.stride = g.stride; A.OH = g.out_h; A.OW = g.out_w;
    } else if (l > 0 && p->layers[l - 1].g.kind == ACTORQ_CONV2D) {
      const LayerGeom &gp = p->layers[l - 1].g;
      A.C = gp.out_c; A.H = gp.out_h; A.W = gp.out_w; A.stride = 1; A.OH = 1; A.OW = 1;
    } else {
      A.C = g.K; A.H = 1; A.W = 1; A.stride = 1; A.OH = 1; A.OW = 1;   // C: bytes between rows
    }
    A.K = g.K; A.Kpad = cg_round_up(g.K, 32); A.nkb = (g.K + 127) / 128;
    A.N = g.N; A.Npad = cg_round_up(g.N, 16); A.nchunk = (A.Npad + kChunkN - 1) / kChunkN;
    A.M = batch * A.OH * A.OW;
    const long long n_tiles = (A.M + kTileM - 1) / kTileM;
    // few row tiles: spread the column chunks over CTAs too; otherwise one CTA keeps all chunks
    A.cpg = (n_tiles >= p->sm_count) ? (A.nchunk < 4 ? A.nchunk : 4) : 1;
    A.n_groups = (A.nchunk + A.cpg - 1) / A.cpg;
    A.acc_bufs = (A.cpg * kChunkN <= 256) ? 2 : 1;
    A.n_items = n_tiles * A.n_groups;
    A.n_a = 6; A.n_b = 4;
    A.in = cur;
    A.koff = L.koff;
    A.n_koff = conv_gemm_koff_entries(p, l);
    A.img = L.wq_img;
    A.colconst = L.colconst;
    if (g.per_channel) { A.ch_zw = L.ch_zw; A.ch_M = L.ch_M; A.ch_P = L.ch_P; }
    A.params = p->d_params;
    A.layer = l; A.last = last ? 1 : 0; A.head = p->head;
    A.out_act = last ? nullptr : bufs[l & 1];
    if (l + 1 == l_tail && l_tail < p->n_layers) {
      A.blk_out = blk;
      A.blk_rs = blk_rs;
      A.blk_nkb = blk_nkb;
      A.blk_unsigned = (p->act[l_tail].z == -128) ? 1 : 0;      // the layer kernel multiplies post-ReLU codes as unsigned bytes
    }
    A.out = last ? out : nullptr;
    A.actions = actions;
    A.out_elems = g.out_elems;
    A.dbg_acc = (l == dbg_layer) ? dbg_acc : nullptr;
    A.dbg_act = (l == dbg_layer && !last) ? dbg_act : nullptr;
    A.status = p->d_status;
    const int smem_bytes = (A.n_a + A.n_b) * kStageBytes + (int)sizeof(ConvGemmBarriers) + A.n_koff * (int)sizeof(int);
    if (smem_bytes > kMaxSmem) return ACTORQ_ERR_UNSUPPORTED;
    const int grid = (int)(A.n_items < p->sm_count ? A.n_items : p->sm_count);
    {   // programmatic dependent launch: the kernel's set-up overlaps the tail of the launch before it
      cudaLaunchConfig_t cfg;
      memset(&cfg, 0, sizeof(cfg));
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.gridDim = dim3((unsigned)grid);
      cfg.blockDim = dim3(kCgThreads);
      cfg.dynamicSmemBytes = (size_t)smem_bytes;
      cfg.stream = st;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      if (cudaLaunchKernelEx(&cfg, conv_gemm_kernel, A) != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_CUDA; }
    }
    p->launches++;
    cur = A.out_act;
  }
  if (l_tail < p->n_layers) return fc_tail_run(p, l_tail, batch, out, actions, dbg_layer, dbg_acc, dbg_act, st);
  return cuda_ok(cudaGetLastError());
}

}  // namespace actorq
