// Wide fully-connected policies, one launch per layer, on CTA pairs (sm_100a, tcgen05
// cta_group::2): the forward pass of policies whose layers are too wide for the fused kernels
// to keep a tile's activations on chip, e.g. the 2048-wide actor networks of the paper's ActorQ
// experiments (Section 3.1: actor inference with the quantized policy; Section 3.2: int8 weights
// and activations; Eq. 3 for the head).
//
// Between layers the int8 activations live in device memory as ready-made MMA operands: for every
// tile of 128 observations and every 128 bytes of K one 16 KB block in the K-major 128-byte-swizzled
// layout, written by the epilogue of the layer before (or by the input quantizer).  A layer is then
// a plain GEMM whose two operands both arrive by bulk copies:
//   raw[256 x n] = A[256 x K] * W[n x K]^T        tcgen05.mma.cta_group::2.kind::i8, n <= 256
// Work item = tile pair (256 observations) x 256 output columns.  Each CTA of the pair stages its own
// 128 rows of A and its half of the n weight rows per K block (32 KB ring stages), one thread of
// the even CTA issues the MMAs for both, and the two 256-column accumulators in tensor memory
// alternate between items, so the epilogue (requantize, Eq. 2 with the ReLU floor, or the head)
// of one item runs under the MMAs of the next.
//
// Row sums: acc = raw + cc[n] - z_w * sum_k a[row][k] needs the sum of a row's stored codes over
// the WHOLE previous layer, whose columns were produced by several items; each epilogue thread adds
// its part to a per-row counter in device memory.  Three counter arrays rotate: layer l reads
// set l % 3, accumulates into set (l + 1) % 3 and clears set (l + 2) % 3 for the layer after.
//
// Codes of a layer whose input zero-point is -128 are kept unsigned (a_u = a_q + 128, u8 x s8 MMA),
// as in the fused pair kernel.  Per-channel layers (their own instantiation) read a zero-point and
// a multiplier per column.  An epilogue warp writes its 32 codes of a row as one 32-byte store, fetches
// the next item's column constants (through 512 bytes of shared memory of its own) and row sum one
// item ahead, and steps through its items without divisions; the head's fp32 tiles leave through
// shared memory so that row segments are written coalesced.  The launches of one forward are
// programmatic dependents of one another: a layer's set-up overlaps the tail of the layer before it.
// Every wait is bounded; a wait that runs out raises ACTORQ_ERR_TIMEOUT and the abort flag of both CTAs.
#include <new>
#include "tcgen05.cuh"

namespace actorq {

namespace fcp {

constexpr int kEpiWarp0 = 2;
constexpr int kEpiWarps = 8;           // two per lane quarter
constexpr int kThreads = (kEpiWarp0 + kEpiWarps) * 32;     // warp 0 producer, 1 issuer / relay, the rest epilogue
constexpr int kAccCols = 256;
constexpr int kPartCols = kAccCols / (kEpiWarps / 4);      // accumulator columns per epilogue warp
constexpr int kPartSlices = kPartCols / 32;
constexpr int kStage = 2 * kStageBytes;    // A block + this CTA's half of the B block
constexpr int kMaxStages = 6;

struct Args {
  const int8_t *a_img;     // input operand blocks  [tile][nkb][16 KB]
  int8_t *out_img;         // output operand blocks [tile][nkb_out][16 KB] (hidden layers)
  const int8_t *w_img;     // weight image: [128-row tile][nkb][16 KB]
  const int *cc;           // per-column constant: bias_q (unsigned input codes) or colconst
  const int *ch_zw;        // per-channel layers (Section 3.2, per-channel quantization): each column's weight
  const float *ch_M;       // zero-point, requantization multiplier and accumulator unit, zero-padded to a
  const float *ch_P;       // multiple of 128 entries; all nullptr for a per-tensor layer
  const int *rs_in;        // per-row sum of the input codes
  int *rs_out;             // per-row sum of the output codes (accumulated)
  int *rs_clear;           // cleared for the next layer
  long long rs_len;
  const LayerParams *params;
  int layer;
  int K, N, Kpad, Npad, nkb, nchunk, nkb_out;
  int chunk_cols;          // output columns per work item: 256, or 128 / 64 when a layer has fewer items than CTA pairs

  int a_unsigned, out_unsigned;
  int last, head;
  int reverse;             // walk the tile pairs from the last one down: the layer before wrote those last, they are the ones still in L2
  long long batch, n_tile_pairs, n_items;
  float *out;
  int *actions;
  const float *sigma;      // exploration noise (tanh heads): per-row sigma and draws, or nullptr
  const float *noise;
  int n_stages;
  int *dbg_acc;            // this layer's accumulators / output codes, or nullptr
  int8_t *dbg_act;
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

template <int V> struct PathC { static constexpr int value = V; };

// kDbg: the instantiation with the debug taps; kPC: the one for per-channel layers (its own copy, so
// that the per-tensor epilogue keeps its registers).
template <bool kDbg, bool kPC>
__global__ void __launch_bounds__(kThreads, 1)
fc_pair_kernel(const __grid_constant__ Args A) {
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {      // (the same in both CTAs of a pair, so both leave)
    if (threadIdx.x == 0) atomicMax(A.status, (int)ACTORQ_ERR_CUDA);
    return;
  }
  uint8_t *ring = smem;
  Barriers *bars = reinterpret_cast<Barriers *>(ring + A.n_stages * kStage);
  int4 *cc_smem = reinterpret_cast<int4 *>(bars + 1);       // [epilogue warp][32]: column constants of the warp's columns

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
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(&bars->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();        // both CTAs' barriers exist before anyone arrives remotely
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  // Launched as a programmatic dependent: everything above overlaps the tail of the previous launch;
  // nothing below runs before that launch has completed (it may still be reading the counters cleared
  // next, and it writes this layer's input).
  griddep_launch_dependents();
  griddep_wait();
  // counters of the layer after the next one's input: cleared here, accumulated by the next launch
  if (A.rs_clear != nullptr)
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < A.rs_len; i += (long long)gridDim.x * kThreads)
      A.rs_clear[i] = 0;
  // A role walks items pair_idx, pair_idx + n_pairs, ..; item = tp * nchunk + c is kept as (tp, c) and
  // stepped without divisions
  const long long tp_first = pair_idx / A.nchunk, tp_step = n_pairs / A.nchunk;
  const int c_first = (int)(pair_idx - tp_first * A.nchunk), c_step = (int)(n_pairs - tp_step * A.nchunk);

  if (warp == 0) {
    // ---------------- producer: this CTA's A rows and its half of the weight rows ----------------
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    long long tp = tp_first;
    int c = c_first;
    for (long long item = pair_idx; item < A.n_items && ok; item += n_pairs) {
      const long long tile = 2 * (A.reverse ? A.n_tile_pairs - 1 - tp : tp) + rank;
      const int rows_c = min(A.chunk_cols, A.Npad - c * A.chunk_cols);
      const int half_rows = rows_c >> 1;
      const int n_first = c * A.chunk_cols + (int)rank * half_rows;     // weight rows [n_first, + half_rows)
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
      tp += tp_step; c += c_step;
      if (c >= A.nchunk) { c -= A.nchunk; ++tp; }
    }
    if (!ok) {   // leave time for bulk copies still in flight into this CTA's shared memory
      for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
  } else if (warp == 1 && rank == 0) {
    // ---------------- MMA issuer (even CTA) ----------------
    int s = 0;
    uint32_t ph = 0, it = 0;
    const uint32_t ring_base = smem_u32(ring);
    bool ok = true;
    int c = c_first;
    for (long long item = pair_idx; item < A.n_items && ok; item += n_pairs, ++it) {
      const int rows_c = min(A.chunk_cols, A.Npad - c * A.chunk_cols);
      c += c_step;
      if (c >= A.nchunk) c -= A.nchunk;
      const uint32_t idesc = instr_desc_pair(rows_c, A.a_unsigned != 0);
      const uint32_t buf = it & 1, use = it >> 1;
      const uint32_t d_tmem = tmem + buf * kAccCols;
      ok = mbar_wait_warp_cl(&bars->acc_empty[buf], (use & 1) ^ 1, abort_flag, peer_abort, A.status);
      if (!ok) break;
      tc_fence_after();
      for (int kb = 0; kb < A.nkb; ++kb) {
        ok = mbar_wait_warp_cl(&bars->ring_full[s], ph, abort_flag, peer_abort, A.status);
        if (!ok) break;
        tc_fence_after();
        const int ksteps = min(128, A.Kpad - kb * 128) >> 5;
        const uint32_t a_lo = desc_lo(ring_base + s * kStage);
        const uint32_t b_lo = desc_lo(ring_base + s * kStage + kStageBytes);
        if (elect_one()) {
          if (ksteps == 4) {
            mma2x4_i8_ss(d_tmem, a_lo, b_lo, kDescHi, idesc, kb != 0);
          } else {
            const uint64_t adesc = ((uint64_t)kDescHi << 32) | a_lo, bdesc = ((uint64_t)kDescHi << 32) | b_lo;
            for (int ks = 0; ks < ksteps; ++ks)
              mma2_i8(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), idesc, (kb | ks) != 0);
          }
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
    const int part = ew >> 2;                  // which kPartCols columns of the 256-column accumulator
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t acc_empty_leader = mapa_u32(smem_u32(&bars->acc_empty[0]), 0);
    const LayerParams p = A.params[A.layer];
    const float hi_f = (float)(127 - p.z_out);
    // hidden layers: FMA-pipe requantization to unsigned codes when the output zero-point is -128
    // and the accumulator / multiplier bounds of requant32_u8 hold; otherwise the exact conversions
    const bool out_u8 = A.out_unsigned != 0;
    const bool fast_u8 = out_u8 && (p.M >= 0x1p-15f) && ((long long)A.K * 65025 + p.bias_absmax < (1ll << 29));
    const bool has_cc = !A.a_unsigned || p.bias_absmax != 0;
    const float Ms = p.M * 0x1p-8f, cs = -8388608.0f * Ms;
    uint32_t it = 0;
    bool ok = true;
    // The row sum of an item's input row and the column constants of its kPartCols columns (one int4
    // per lane) are fetched one item ahead; the constants then go through this warp's own 512 bytes
    // of shared memory, from where the requantizer reads them as broadcasts.
    int4 *cc_warp = cc_smem + ew * 32;
    float *head_buf = reinterpret_cast<float *>(cc_smem + kEpiWarps * 32);     // 16 KB: the head's output tiles
    long long tp = tp_first, tp_nx;
    int c = c_first, c_nx;
    auto step = [&](long long t, int cc, long long &t2, int &c2) {
      t2 = t + tp_step; c2 = cc + c_step;
      if (c2 >= A.nchunk) { c2 -= A.nchunk; ++t2; }
    };
    auto fetch_rs = [&](long long t) { return __ldg(A.rs_in + (2 * (A.reverse ? A.n_tile_pairs - 1 - t : t) + rank) * kTileM + row); };
    auto fetch_cc = [&](int cc) {     // (the array is zero-padded to a multiple of 128 entries; chunks may end earlier)
      const int n = cc * A.chunk_cols + part * kPartCols + 4 * lane;
      return (n < ((A.N + 127) & ~127)) ? __ldg(reinterpret_cast<const int4 *>(A.cc + n)) : make_int4(0, 0, 0, 0);
    };
    int rs_next = 0;
    int4 cc_next = make_int4(0, 0, 0, 0);
    if (pair_idx < A.n_items) { rs_next = fetch_rs(tp); cc_next = fetch_cc(c); }
    for (long long item = pair_idx; item < A.n_items && ok; item += n_pairs, ++it, tp = tp_nx, c = c_nx) {
      step(tp, c, tp_nx, c_nx);
      const long long tile = 2 * (A.reverse ? A.n_tile_pairs - 1 - tp : tp) + rank;
      const long long grow = tile * kTileM + row;
      const bool row_valid = grow < A.batch;
      const int rs_in = rs_next;
      __syncwarp();                       // every lane is done with the previous item's constants
      cc_warp[lane] = cc_next;
      __syncwarp();
      if (item + n_pairs < A.n_items) { rs_next = fetch_rs(tp_nx); cc_next = fetch_cc(c_nx); }
      const int rows_c = min(A.chunk_cols, A.Npad - c * A.chunk_cols);
      const uint32_t buf = it & 1, use = it >> 1;
      const uint32_t acc = tmem + lane_addr + buf * kAccCols;
      const int rterm = -p.z_w * rs_in;
      const float sigma_row = (A.last && A.noise != nullptr && row_valid) ? __ldg(A.sigma + grow) : 0.0f;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_full[buf], use & 1, abort_flag, A.status));
      if (!ok) break;
      tc_fence_after();
      if (!A.last) {
        // ---- hidden layer: this warp requantizes columns [kPartCols part, +kPartCols) of the item for its 32 rows
        // and writes them as 16-byte pieces of the next layer's operand blocks ----
        int rowsum_out = 0;
        const int n_slices = min(kPartSlices, max(0, (rows_c - part * kPartCols + 31) / 32));
        // one copy of the four-slice loop per requantize path (0: FMA pipe, 1: the same plus a column
        // constant, 2: exact conversions), so that the path taken is one contiguous run of code
        // (64 columns per tensor-memory load; after the last one the accumulator goes back to the MMA issuer)
        auto slices = [&](auto path) {
          constexpr int kPath = decltype(path)::value;
        uint32_t r64[64];
        const uint32_t (&rr)[2][32] = *reinterpret_cast<const uint32_t (*)[2][32]>(&r64);
        if (n_slices == 0) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8u * buf);
        }
#pragma unroll
        for (int s = 0; s < kPartSlices; ++s) {
          if (s >= n_slices) break;
          const int col0 = part * kPartCols + s * 32;
          if ((s & 1) == 0) {
            tmem_ld64_wait(acc + col0, r64);
            if (s + 2 >= n_slices) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8u * buf);
            }
          }
          const uint32_t (&r)[32] = rr[s & 1];
          const int n0 = c * A.chunk_cols + col0;
          const int4 *cc4 = cc_warp + s * 8;
          uint32_t packed[8];
          if (kPath == 0) requant32_u8<false>(r, cc4, (uint32_t)rterm + 0x4B000000u, Ms, cs, packed);
          else if (kPath == 1) {
            int4 ccr[8];                     // the slice's constants: all eight loads in flight together
#pragma unroll
            for (int j = 0; j < 8; ++j) ccr[j] = cc4[j];
            requant32_u8<true>(r, ccr, (uint32_t)rterm + 0x4B000000u, Ms, cs, packed);
          }
          else if (kPath == 3) {       // per-channel: column n has its own z_w[n] and M[n]
            requant32_pc(r, A.cc + n0, A.ch_zw + n0, A.ch_M + n0, rs_in, hi_f, p.z_out, packed);
            if (out_u8) {
#pragma unroll
              for (int j = 0; j < 8; ++j) packed[j] ^= 0x80808080u;
            }
          } else {
            requant32<0, true>(r, cc4, rterm, p.M, hi_f, p.z_out, packed);       // signed codes
            if (out_u8) {
#pragma unroll
              for (int j = 0; j < 8; ++j) packed[j] ^= 0x80808080u;
            }
          }
          if (kDbg && A.dbg_acc != nullptr && row_valid) {
            for (int j = 0; j < 32; ++j)
              if (n0 + j < A.N)
                A.dbg_acc[grow * A.N + n0 + j] =
                    (int)(r[j] + (uint32_t)__ldg(A.cc + n0 + j) + (uint32_t)(kPC ? -__ldg(A.ch_zw + n0 + j) * rs_in : rterm));
          }
          if (n0 + 32 > A.N) {                                 // K padding of the next layer: code 0
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              uint32_t keep = 0;
#pragma unroll
              for (int e = 0; e < 4; ++e) if (n0 + 4 * j + e < A.N) keep |= 0xffu << (8 * e);
              packed[j] &= keep;
            }
          }
          if (out_u8) {
#pragma unroll
            for (int j = 0; j < 8; ++j) rowsum_out = (int)__dp4a(packed[j], 0x01010101u, (unsigned)rowsum_out);
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) rowsum_out = __dp4a((int)packed[j], 0x01010101, rowsum_out);
          }
          if (kDbg && A.dbg_act != nullptr && row_valid) {     // the int8 code of an unsigned byte n is n - 128
            for (int j = 0; j < 32; ++j)
              if (n0 + j < A.N) A.dbg_act[grow * A.N + n0 + j] = (int8_t)((packed[j >> 2] >> (8 * (j & 3))) ^ (out_u8 ? 0x80u : 0u));
          }
          const uint32_t kc = ((uint32_t)n0 & 127) >> 4;       // 16-byte column of the first 16 codes
          int8_t *rowp = A.out_img + (((size_t)tile * A.nkb_out + (size_t)(n0 >> 7)) << 14) + ((uint32_t)row << 7);
          // the two 16-byte pieces (kc even) share one aligned 32-byte sector, in swapped order on odd
          // rows of the swizzle: one 32-byte store
          const bool swap = ((uint32_t)row & 1u) != 0;
          st_global_v8(rowp + ((kc ^ ((uint32_t)row & 6)) << 4),
                       swap ? packed[4] : packed[0], swap ? packed[5] : packed[1], swap ? packed[6] : packed[2], swap ? packed[7] : packed[3],
                       swap ? packed[0] : packed[4], swap ? packed[1] : packed[5], swap ? packed[2] : packed[6], swap ? packed[3] : packed[7]);
        }
        };
        if constexpr (kPC) {
          slices(PathC<3>{});
        } else {
          if (fast_u8) { if (has_cc) slices(PathC<1>{}); else slices(PathC<0>{}); }
          else slices(PathC<2>{});
        }
        if (n_slices > 0) atomicAdd(A.rs_out + grow, rowsum_out);
      } else {
        // ---- head: at most 128 columns.  tanh / linear heads: the two warps of a lane quarter take 16
        // columns each of every 32; a greedy-action head is done by the part-0 warps alone (one
        // running maximum per row); warps of later parts only hand the accumulator back ----
        const bool split = (A.head != ACTORQ_HEAD_ARGMAX);
        const int n_slices = (part == 0 || (split && part == 1)) ? (rows_c + 31) / 32 : 0;
        const int sub = split ? part * 16 : 0;
        float best_v = 0.0f;
        int best_n = -1;
        if (n_slices == 0) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8u * buf);
        }
        // (every column of the slice is computed, without branches, so that the tanh chains of a thread's
        // columns overlap; columns past N only never leave: the constant arrays are zero-padded)
        auto head_slice = [&](auto width, int col0, bool last_slice) {
          constexpr int kW = decltype(width)::value;          // columns per thread: 16 (split) or 32
          uint32_t r[32];
          tmem_ld32_wait(acc + col0, r);                      // (a split warp uses the first 16 of them)
          if (last_slice) {                                   // the accumulator goes back before the arithmetic
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8u * buf);
          }
          const int n0 = col0;
          int ccv[kW];
#pragma unroll
          for (int j4 = 0; j4 < kW / 4; ++j4) {
            const int4 cc = __ldg(reinterpret_cast<const int4 *>(A.cc + n0) + j4);
            ccv[4 * j4] = cc.x; ccv[4 * j4 + 1] = cc.y; ccv[4 * j4 + 2] = cc.z; ccv[4 * j4 + 3] = cc.w;
          }
          float y[kW];
#pragma unroll
          for (int j = 0; j < kW; ++j) {
            const int av = (int)(r[j] + (uint32_t)ccv[j] + (uint32_t)(kPC ? -__ldg(A.ch_zw + n0 + j) * rs_in : rterm));
            if (kDbg && A.dbg_acc != nullptr && row_valid && n0 + j < A.N) A.dbg_acc[grow * A.N + n0 + j] = av;
            y[j] = __fmul_rn(__int2float_rn(av), kPC ? __ldg(A.ch_P + n0 + j) : p.P);          // Eq. 3 on the accumulator
          }
          if (A.head == ACTORQ_HEAD_ARGMAX) {
#pragma unroll
            for (int j = 0; j < kW; ++j)
              if (n0 + j < A.N && (y[j] > best_v || best_n < 0)) { best_v = y[j]; best_n = n0 + j; }
          } else if (A.head == ACTORQ_HEAD_TANH) {
#pragma unroll
            for (int j = 0; j < kW; ++j) y[j] = tanhf(y[j]);
            if (A.noise != nullptr && row_valid) {            // actor exploration: y + sigma * eps, kept in [-1, 1]
#pragma unroll
              for (int j = 0; j < kW; ++j)
                if (n0 + j < A.N) {
                  const float t = __fadd_rn(y[j], __fmul_rn(sigma_row, __ldg(A.noise + grow * A.N + n0 + j)));
                  y[j] = fminf(fmaxf(t, -1.0f), 1.0f);
                }
            }
          }
#pragma unroll
          for (int j = 0; j < kW; ++j) r[j] = __float_as_uint(y[j]);
          // the warp's 32 rows x 16 (32) columns leave through shared memory, row segments coalesced
          const long long wrow0 = tile * kTileM + quarter * 32;
          const int rows_valid = (int)max(0ll, min(32ll, A.batch - wrow0));
          warp_store_rows<kW>(A.out, wrow0, rows_valid, A.N, n0, r, head_buf + ew * (32 * kW), lane);
        };
        for (int s = 0; s < n_slices; ++s) {
          if (split) head_slice(PathC<16>{}, s * 32 + sub, s + 1 == n_slices);
          else head_slice(PathC<32>{}, s * 32, s + 1 == n_slices);
        }
        if (A.head == ACTORQ_HEAD_ARGMAX && part == 0 && row_valid) A.actions[grow] = best_n;
      }
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

// Input quantizer (Eq. 1 on the observations): float rows [batch][K] -> the first layer's operand
// blocks and the per-row sums of the codes; also clears the counters the first layer accumulates into.
// One block per tile of 128 rows; thread = (row, one of up to four 32-column slices it strides over).
__global__ void __launch_bounds__(512)
quantize_obs_blocks_kernel(const float *__restrict__ obs, long long batch, long long rows_pad, int K, int nkb,
                           const LayerParams *__restrict__ params, int8_t *__restrict__ img, int *__restrict__ rs0,
                           int *__restrict__ rs1) {
  __shared__ int rowsum[128];
  const LayerParams p0 = params[0];
  const int r = threadIdx.x & 127, sl = threadIdx.x >> 7, n_sl = blockDim.x >> 7;
  const long long grow = (long long)blockIdx.x * 128 + r;
  if (sl == 0) rowsum[r] = 0;
  __syncthreads();
  const bool r_ok = grow < batch;
  const bool vec_ok = ((K & 3) == 0) && ((reinterpret_cast<uintptr_t>(obs) & 15) == 0);
  const float lo_f = (float)(-128 - p0.z_a), hi_f = (float)(127 - p0.z_a);
  const float *xrow = obs + (r_ok ? grow : batch - 1) * K;
  uint8_t *a0 = reinterpret_cast<uint8_t *>(img) + (((size_t)blockIdx.x * nkb) << 14);
  int rsum = 0;
  for (int k0 = sl * 32; k0 < K; k0 += n_sl * 32) rsum += quantize_obs32(xrow, K, vec_ok, k0, r_ok, r, p0.inv_s_a, p0.z_a, lo_f, hi_f, a0);
  atomicAdd(&rowsum[r], rsum);
  __syncthreads();
  if (sl == 0 && grow < rows_pad) {
    rs0[grow] = rowsum[r];
    rs1[grow] = 0;
  }
}

}  // namespace fcp

// ---- host side ------------------------------------------------------------------------------

static int fcp_round_up(int v, int m) { return (v + m - 1) / m * m; }

bool fc_pair_supported(const actorq_policy *p) {
  if (p->obs_dtype != ACTORQ_OBS_F32 || p->n_layers < 2) return false;
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerGeom &g = p->layers[l].g;
    const bool last = (l + 1 == p->n_layers);
    if (g.kind != ACTORQ_FC) return false;
    if (last ? g.N > 128 : g.N > 8192) return false;
  }
  return true;
}

// bytes of one activation buffer per padded row: the widest layer input, in whole 128-byte K blocks
static long long fcp_row_bytes(const actorq_policy *p) {
  int kmax = 0;
  for (int l = 0; l < p->n_layers; ++l) kmax = p->layers[l].g.K > kmax ? p->layers[l].g.K : kmax;
  return fcp_round_up(kmax, 128);
}

static int fcp_ensure(actorq_policy *p, long long rows_pad) {
  if (rows_pad <= p->fcp_rows) return ACTORQ_OK;
  if (p->fcp_mem) cudaFree(p->fcp_mem);
  p->fcp_mem = nullptr;
  p->fcp_rows = 0;
  const size_t one = (size_t)rows_pad * (size_t)fcp_row_bytes(p);
  void *mem = nullptr;
  if (cudaMalloc(&mem, 2 * one + 3 * (size_t)rows_pad * sizeof(int)) != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_NOMEM; }
  p->fcp_mem = mem;
  p->fcp_rows = rows_pad;
  return ACTORQ_OK;
}

struct FcpLaunch {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  int max_pairs;
  int n_stages;
  long long n_tile_pairs, rows_pad;
  int8_t *bufs[2];
  int *rs[3];
};

// Launch configuration, activation buffers and row-sum arrays for `batch` rows.
static int fcp_prepare(actorq_policy *p, long long batch, cudaStream_t st, FcpLaunch &F) {
  static bool attr_set[64] = {false};
  static int max_clusters[64] = {0};
  const int dev = p->device;
  if (dev < 0 || dev >= 64) return ACTORQ_ERR_UNSUPPORTED;
  const int n_stages = fcp::kMaxStages;
  const int smem_bytes = n_stages * fcp::kStage + (int)sizeof(fcp::Barriers) + fcp::kEpiWarps * 32 * (int)sizeof(int4) + 16384;
  if (smem_bytes > kMaxSmem) return ACTORQ_ERR_UNSUPPORTED;
  cudaLaunchConfig_t &cfg = F.cfg;
  cudaLaunchAttribute *attr = F.attr;
  memset(&cfg, 0, sizeof(cfg));
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.blockDim = dim3(fcp::kThreads);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(fcp::fc_pair_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess ||
        cudaFuncSetAttribute(fcp::fc_pair_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess ||
        cudaFuncSetAttribute(fcp::fc_pair_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess ||
        cudaFuncSetAttribute(fcp::fc_pair_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
      return ACTORQ_ERR_CUDA;
    cfg.gridDim = dim3((unsigned)(p->sm_count & ~1));
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, fcp::fc_pair_kernel<false, false>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
    max_clusters[dev] = n;
    attr_set[dev] = true;
  }
  if (max_clusters[dev] < 1) return ACTORQ_ERR_UNSUPPORTED;

  const long long n_tiles = (batch + kTileM - 1) / kTileM;
  const long long n_tile_pairs = (n_tiles + 1) / 2;
  const long long rows_pad = n_tile_pairs * 2 * kTileM;
  const int rc = fcp_ensure(p, rows_pad);
  if (rc != ACTORQ_OK) return rc;
  const size_t one = (size_t)p->fcp_rows * (size_t)fcp_row_bytes(p);
  F.bufs[0] = (int8_t *)p->fcp_mem;
  F.bufs[1] = (int8_t *)p->fcp_mem + one;
  F.rs[0] = reinterpret_cast<int *>((int8_t *)p->fcp_mem + 2 * one);
  F.rs[1] = F.rs[0] + p->fcp_rows;
  F.rs[2] = F.rs[1] + p->fcp_rows;
  F.max_pairs = max_clusters[dev];
  F.n_stages = n_stages;
  F.n_tile_pairs = n_tile_pairs;
  F.rows_pad = rows_pad;
  return ACTORQ_OK;
}

// Layers [l_begin, n_layers) on the layer kernel.  Layer l reads the operand blocks in bufs[l & 1] and
// the row sums in rs[l % 3]; whoever fills them for l_begin has also left rs[(l_begin + 1) % 3] zeroed.
static int fcp_run_layers(actorq_policy *p, FcpLaunch &F, int l_begin, long long batch, float *out, int *actions,
                          int dbg_layer, int *dbg_acc, int8_t *dbg_act) {
  cudaLaunchConfig_t &cfg = F.cfg;
  int8_t **bufs = F.bufs;
  int **rs = F.rs;
  const long long n_tile_pairs = F.n_tile_pairs, rows_pad = F.rows_pad;
  const int n_stages = F.n_stages;
  for (int l = l_begin; l < p->n_layers; ++l) {
    const LayerDev &L = p->layers[l];
    const bool last = (l + 1 == p->n_layers);
    fcp::Args A;
    memset(&A, 0, sizeof(A));
    A.a_img = bufs[l & 1];
    A.out_img = last ? nullptr : bufs[(l + 1) & 1];
    A.w_img = L.wq_img;
    A.a_unsigned = (l > 0 && p->act[l].z == -128) ? 1 : 0;
    A.out_unsigned = (!last && p->act[l + 1].z == -128) ? 1 : 0;
    A.cc = A.a_unsigned ? L.bias_q : L.colconst;
    if (L.g.per_channel) { A.ch_zw = L.ch_zw; A.ch_M = L.ch_M; A.ch_P = L.ch_P; }
    A.rs_in = rs[l % 3];
    A.rs_out = rs[(l + 1) % 3];
    A.rs_clear = (l + 2 < p->n_layers) ? rs[(l + 2) % 3] : nullptr;
    A.rs_len = rows_pad;
    A.params = p->d_params;
    A.layer = l;
    A.K = L.g.K;
    A.N = L.g.N;
    A.Kpad = fcp_round_up(L.g.K, 32);
    A.Npad = fcp_round_up(L.g.N, 32);
    A.nkb = (L.g.K + 127) / 128;
    // a layer with fewer (tile pair, 256 columns) items than CTA pairs is cut into narrower items: more
    // pairs work, and an item's K loop is shorter per MMA (a K loop cannot be shorter than its MMA count)
    A.chunk_cols = fcp::kAccCols;
    while (A.chunk_cols > 64 && !last && n_tile_pairs * ((A.Npad + A.chunk_cols - 1) / A.chunk_cols) < F.max_pairs) A.chunk_cols >>= 1;
    A.nchunk = (A.Npad + A.chunk_cols - 1) / A.chunk_cols;
    A.nkb_out = (L.g.N + 127) / 128;
    A.last = last ? 1 : 0;
    A.reverse = (l - l_begin) & 1;       // alternate directions: a layer starts where the one before it ended
    A.head = p->head;
    A.batch = batch;
    A.n_tile_pairs = n_tile_pairs;
    A.n_items = n_tile_pairs * A.nchunk;
    A.out = out;
    A.actions = actions;
    if (last && p->ex_noise != nullptr && p->head == ACTORQ_HEAD_TANH && dbg_layer < 0) {
      A.sigma = p->ex_sigma;
      A.noise = p->ex_noise;
      p->ex_applied = 1;
    }
    A.n_stages = n_stages;
    A.dbg_acc = (l == dbg_layer) ? dbg_acc : nullptr;
    A.dbg_act = (l == dbg_layer && !last) ? dbg_act : nullptr;
    A.status = p->d_status;
    const long long pairs = A.n_items < F.max_pairs ? A.n_items : F.max_pairs;
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.numAttrs = 2;          // clusters of two + programmatic dependent launch
    const bool pc = L.g.per_channel != 0;
    const cudaError_t e = (l == dbg_layer) ? (pc ? cudaLaunchKernelEx(&cfg, fcp::fc_pair_kernel<true, true>, A)
                                                 : cudaLaunchKernelEx(&cfg, fcp::fc_pair_kernel<true, false>, A))
                                           : (pc ? cudaLaunchKernelEx(&cfg, fcp::fc_pair_kernel<false, true>, A)
                                                 : cudaLaunchKernelEx(&cfg, fcp::fc_pair_kernel<false, false>, A));
    p->launches++;
    if (e != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_CUDA; }
  }
  return ACTORQ_OK;
}

int launch_forward_fc_pair(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                           int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st) {
  if (!p->fcp_ok) return ACTORQ_ERR_UNSUPPORTED;
  for (int l = 0; l < p->n_layers; ++l)
    if (p->layers[l].wq_img == nullptr) return ACTORQ_ERR_UNSUPPORTED;
  FcpLaunch F;
  const int rc = fcp_prepare(p, batch, st, F);
  if (rc != ACTORQ_OK) return rc;
  const int K0 = p->layers[0].g.K;
  const int obs_slices = (K0 + 31) / 32 < 4 ? (K0 + 31) / 32 : 4;
  fcp::quantize_obs_blocks_kernel<<<(unsigned)(F.rows_pad / 128), 128 * obs_slices, 0, st>>>((const float *)obs, batch, F.rows_pad, K0, (K0 + 127) / 128,
                                                                               p->d_params, F.bufs[0], F.rs[0], F.rs[1]);
  p->launches++;
  return fcp_run_layers(p, F, 0, batch, out, actions, dbg_layer, dbg_acc, dbg_act);
}

// The fully connected tail of a convolutional policy (layers l_begin .. n_layers - 1) on the layer
// kernel.  fc_tail_begin hands out where the kernel of layer l_begin - 1 must leave its output: operand
// blocks (one 16 KB block [128 rows][128 B], 128-byte swizzle, per 128-row tile and 128 bytes of the
// row) and per-row sums of the codes, accumulated with atomic adds into an array zeroed here.
// clear_here: zero the row-sum arrays with a memset on the stream; otherwise the caller has a kernel
// that runs before the accumulating one clear [*rs_all, *rs_all + *rs_all_len).
int fc_tail_begin(actorq_policy *p, int l_begin, long long batch, cudaStream_t st, int8_t **blocks, int *nkb, int **rowsums,
                  int clear_here, int **rs_all, long long *rs_all_len) {
  if (l_begin < 1 || l_begin >= p->n_layers) return ACTORQ_ERR_UNSUPPORTED;
  for (int l = l_begin; l < p->n_layers; ++l) {
    const LayerGeom &g = p->layers[l].g;
    const bool last = (l + 1 == p->n_layers);
    if (g.kind != ACTORQ_FC || p->layers[l].wq_img == nullptr) return ACTORQ_ERR_UNSUPPORTED;
    if (last ? g.N > 128 : g.N > 8192) return ACTORQ_ERR_UNSUPPORTED;
  }
  FcpLaunch F;
  const int rc = fcp_prepare(p, batch, st, F);
  if (rc != ACTORQ_OK) return rc;
  if (clear_here && cudaMemsetAsync(F.rs[0], 0, 3 * (size_t)p->fcp_rows * sizeof(int), st) != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_CUDA; }
  *rs_all = F.rs[0];
  *rs_all_len = 3 * p->fcp_rows;
  *blocks = F.bufs[l_begin & 1];
  *nkb = (p->layers[l_begin].g.K + 127) / 128;
  *rowsums = F.rs[l_begin % 3];
  return ACTORQ_OK;
}

int fc_tail_run(actorq_policy *p, int l_begin, long long batch, float *out, int *actions,
                int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st) {
  FcpLaunch F;
  const int rc = fcp_prepare(p, batch, st, F);
  if (rc != ACTORQ_OK) return rc;
  return fcp_run_layers(p, F, l_begin, batch, out, actions, dbg_layer, dbg_acc, dbg_act);
}

}  // namespace actorq
