// Fused int8 MLP forward on CTA pairs (sm_100a, tcgen05 cta_group::2): the throughput form of
// the fused kernel in mlp_fused.cu (paper Section 3.1: actor inference with the quantized policy;
// Section 3.2: int8 weights and activations; Eq. 3 for the head).
//
// Two CTAs on neighbouring SMs form a cluster.  Each owns one 128-observation tile (its A operand,
// its accumulators, its epilogue), and one thread of the even CTA issues every MMA for both:
//   raw[256 x n] = A[256 x K] * W[n x K]^T        tcgen05.mma.cta_group::2.kind::i8, n <= 256
// Rows 0..127 of A / raw live in the even CTA, rows 128..255 in the odd one; each CTA stages only
// its half of the n weight rows of a K block (the tensor cores exchange the halves), so a weight
// byte is fetched from L2 once per 256 observations and a 16 KB ring stage feeds four n = 256
// instructions.  A single thread cannot issue MMAs faster than about one per 60-70 cycles; only
// at n = 256 (128 cycles of arithmetic per instruction) does the issue rate stop being the limit.
//
// Tensor memory per CTA: columns 0..255 one accumulator of up to 256 output columns, columns
// 256..511 the A operand of layers 1, 3, ..  The accumulator is single-buffered: the epilogue warps
// pull their 128 columns into registers in one load and hand it back before they start the
// arithmetic, so the MMA stream pauses only for that load.  As in the single-CTA kernel the A
// operand alternates between tensor memory and shared memory, and output chunk c (256 columns)
// is K blocks 2c, 2c+1 of the next layer, released as soon as it is written.
//
// Barriers: waits of the issuing thread use the EVEN CTA's barriers, on which threads of both CTAs
// arrive (remote arrives through shared::cluster addresses); completions of the issuer
// (tcgen05.commit) arrive on the same barrier in both CTAs.  The odd CTA's MMA warp only relays
// "my half of this ring stage has landed" to the even CTA.  Every wait is bounded; a wait that runs
// out raises ACTORQ_ERR_TIMEOUT and the abort flag of both CTAs.
#include <new>
#include "tcgen05.cuh"

namespace actorq {

namespace pair {

constexpr int kThreads = 384;
constexpr int kLoaderWarp0 = 2;
constexpr int kLoaderWarps = 2;
constexpr int kEpiWarp0 = 4;
constexpr int kEpiWarps = 8;
constexpr int kAccCols = 256;          // accumulator columns (one buffer)
constexpr int kActCol = 256;           // TMEM column where the int8 activation operand starts
constexpr int kMaxChunks = 4;          // 256-column chunks per layer (N <= 1024)
constexpr int kMaxStages = 8;
constexpr int kCcEntries = kMaxChunks * kAccCols;

struct Layer {
  const int8_t *img;
  const int *cc;           // per-column integer constant (see a_unsigned), zero-padded to a multiple of 128 entries
  int K, N;
  int Kpad;                // K rounded up to 32 (MMA K step)
  int Npad;                // N rounded up to 32: each CTA supplies Npad/2 weight rows, a multiple of 16
  int nkb;                 // 128-byte K blocks
  int nchunk;              // 256-column chunks
  // The input codes of a layer whose input zero-point is -128 (every layer fed by a ReLU) are kept
  // as UNSIGNED bytes a_u = a_q + 128 and multiplied as such (u8 x s8).  Then
  //   sum_k (a_q - z_a)(w_q - z_w) + bias_q = sum_k a_u w_q - z_w sum_k a_u + bias_q :
  // the per-column constant is the bias alone (cc = bias_q, all zero for a policy without biases)
  // instead of colconst = bias_q - z_a colsum + K z_a z_w (cc = colconst, signed codes).
  int a_unsigned;          // this layer's input codes are unsigned
  int out_unsigned;        // this layer's output codes are unsigned (= a_unsigned of the next layer)
};

struct Args {
  int n_layers;
  Layer L[ACTORQ_MAX_LAYERS];
  const LayerParams *params;
  const float *obs;
  long long batch;
  long long n_tile_pairs;
  float *out;
  int *actions;
  const float *sigma;      // exploration noise (tanh heads): per-row sigma [batch] and draws [batch][out_dim], or nullptr
  const float *noise;
  int head;
  int obs_dim, out_dim;
  int n_stages;
  int abig_bytes, a0_bytes;
  int stages_per_pair;     // ring stages consumed per tile pair (all layers)
  int dbg_layer;           // -1: none
  int *dbg_acc;
  int8_t *dbg_act;
  int *status;
};

struct __align__(16) Barriers {
  uint64_t ring_full[kMaxStages];
  uint64_t ring_empty[kMaxStages];
  uint64_t acc_full;
  uint64_t acc_empty;
  uint64_t a0_full;
  uint64_t a0_first;               // the first tile's observations (loaded by all loader and epilogue warps)
  uint64_t a0_empty;
  uint64_t out_ready[2 * kMaxChunks];   // one per 128 output columns = K block of the next layer
  uint64_t drain;
  uint64_t cc_ready[2];
  uint32_t tmem_base;
  int abort_flag;
};

// The first tile of a CTA has nothing to hide behind: all ten loader / epilogue warps share it, one
// work item = 32 rows x 32 columns, row sums combined with shared-memory atomics (rs0 zeroed before).
__device__ __forceinline__ void load_first_tile(const float *obs, long long batch, long long row0, int K0, int K0pad128,
                                                const LayerParams &p0, uint8_t *a0, int *rowsum0, int helper, int n_helpers,
                                                int lane) {
  const bool vec_ok = ((K0 & 3) == 0) && ((reinterpret_cast<uintptr_t>(obs) & 15) == 0);
  const float lo_f = (float)(-128 - p0.z_a), hi_f = (float)(127 - p0.z_a);
  const int valid = (int)max(0ll, min((long long)kTileM, batch - row0));
  const int kslices = K0pad128 >> 5;
  for (int item = helper; item < 4 * kslices; item += n_helpers) {
    const int r = (item / kslices) * 32 + lane, k0 = (item % kslices) * 32;
    const float *xrow = obs + (valid > 0 ? (row0 + min(r, valid - 1)) * K0 : 0);
    const int rsum = quantize_obs32(xrow, K0, vec_ok, k0, r < valid, r, p0.inv_s_a, p0.z_a, lo_f, hi_f, a0);
    atomicAdd(rowsum0 + r, rsum);
  }
}

template <int V> struct PathC { static constexpr int value = V; };

// kDbg: the instantiation with the debug taps (one layer's accumulators and codes written to global
// memory); the production instantiation carries none of that code.
template <bool kDbg>
__global__ void __launch_bounds__(kThreads, 1)
fused_mlp_pair_kernel(const __grid_constant__ Args A) {
  extern __shared__ __align__(1024) uint8_t smem[];
  // (an unaligned dynamic shared memory base would be the same in both CTAs, so both leave)
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0) atomicMax(A.status, (int)ACTORQ_ERR_CUDA);
    return;
  }
  uint8_t *a_big = smem;
  uint8_t *a0 = a_big + A.abig_bytes;
  uint8_t *ring = a0 + A.a0_bytes;
  Barriers *bars = reinterpret_cast<Barriers *>(ring + A.n_stages * kStageBytes);
  int *rs0 = reinterpret_cast<int *>(bars + 1);             // [tile parity][row]
  int *rsp = rs0 + 2 * kTileM;                              // [layer parity][column half][row]
  int4 *cc_smem = reinterpret_cast<int4 *>(rsp + 4 * kTileM);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();                  // 0: issues the MMAs
  const long long pair_idx = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  volatile int *abort_flag = &bars->abort_flag;
  const uint32_t peer_abort = mapa_u32(smem_u32(&bars->abort_flag), rank ^ 1u);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(&bars->ring_full[s], rank == 0 ? 2 : 1);    // own bulk copies (+ the odd CTA's relay)
      mbar_init(&bars->ring_empty[s], 1);
    }
    mbar_init(&bars->acc_full, 1);
    mbar_init(&bars->acc_empty, 2 * kEpiWarps);
    mbar_init(&bars->a0_full, 2 * kLoaderWarps * 32);
    mbar_init(&bars->a0_first, 2 * (kLoaderWarps + kEpiWarps) * 32);
    mbar_init(&bars->a0_empty, 1);
    for (int c = 0; c < 2 * kMaxChunks; ++c) mbar_init(&bars->out_ready[c], 2 * kEpiWarps);
    mbar_init(&bars->drain, 1);
    for (int b = 0; b < 2; ++b) mbar_init(&bars->cc_ready[b], kEpiWarps);
    bars->abort_flag = 0;
    if (blockIdx.x == 0) A.status[7] = (int)smem_u32(bars);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(&bars->tmem_base, 512);
  if (threadIdx.x >= kThreads - kTileM) rs0[threadIdx.x - (kThreads - kTileM)] = 0;   // first tile: atomically accumulated
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();        // both CTAs' barriers exist before anyone arrives remotely
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp < kEpiWarp0) {
  if (warp == 0) {
    // ---------------- weight-ring producer: this CTA's half of every B tile ----------------
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    for (long long tp = pair_idx; tp < A.n_tile_pairs && ok; tp += n_pairs) {
      for (int l = 0; l < A.n_layers && ok; ++l) {
        const Layer &L = A.L[l];
        for (int c = 0; c < L.nchunk && ok; ++c) {
          const int rows_c = min(kAccCols, L.Npad - c * kAccCols);
          const int half_rows = rows_c >> 1;
          // weight rows [n_first, n_first + half_rows) of the layer; image tiles hold 128 rows
          const int n_first = c * kAccCols + (int)rank * half_rows;
          const int t0 = n_first >> 7, r0 = n_first & 127;
          const int rows_a = min(half_rows, 128 - r0);         // rows taken from tile t0
          const int rows_b = half_rows - rows_a;               // rest, from the next tile
          const uint32_t bytes = (uint32_t)half_rows * 128;
          for (int kb = 0; kb < L.nkb; ++kb) {
            ok = mbar_wait_warp(&bars->ring_empty[s], ph ^ 1, abort_flag, A.status);
            if (!ok) break;
            if (elect_one()) {
              uint8_t *dst = ring + s * kStageBytes;
              mbar_expect_tx(&bars->ring_full[s], bytes);
              bulk_g2s(dst, L.img + (((size_t)t0 * L.nkb + kb) << 14) + ((size_t)r0 << 7), (uint32_t)rows_a * 128, &bars->ring_full[s]);
              if (rows_b > 0)
                bulk_g2s(dst + rows_a * 128, L.img + (((size_t)(t0 + 1) * L.nkb + kb) << 14), (uint32_t)rows_b * 128, &bars->ring_full[s]);
            }
            __syncwarp();
            if (++s == A.n_stages) { s = 0; ph ^= 1; }
          }
        }
      }
    }
    if (!ok) {   // leave time for bulk copies still in flight into this CTA's shared memory
      for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
  } else if (warp == 1 && rank == 0) {
    // ---------------- MMA issuer (even CTA) ----------------
    int s = 0;
    uint32_t ph = 0, chunk_ctr = 0, tp_it = 0, ready_bits = 0;
    const uint32_t ring_base = smem_u32(ring);
    bool ok = true;
    for (long long tp = pair_idx; tp < A.n_tile_pairs && ok; tp += n_pairs, ++tp_it) {
      for (int l = 0; l < A.n_layers && ok; ++l) {
        const Layer &L = A.L[l];
        const bool a_in_tmem = (l & 1) != 0;
        const uint32_t a_base = smem_u32(l == 0 ? a0 : a_big);
        if (l == 0) {
          ok = tp_it == 0 ? mbar_wait_warp_cl(&bars->a0_first, 0, abort_flag, peer_abort, A.status)
                          : mbar_wait_warp_cl(&bars->a0_full, (tp_it - 1) & 1, abort_flag, peer_abort, A.status);
          if (!ok) break;
          tc_fence_after();
        }
        for (int c = 0; c < L.nchunk && ok; ++c, ++chunk_ctr) {
          const int rows_c = min(kAccCols, L.Npad - c * kAccCols);
          const uint32_t idesc = instr_desc_pair(rows_c, L.a_unsigned != 0);
          ok = mbar_wait_warp_cl(&bars->acc_empty, (chunk_ctr & 1) ^ 1, abort_flag, peer_abort, A.status);
          if (!ok) break;
          tc_fence_after();
          for (int kb = 0; kb < L.nkb; ++kb) {
            if (l > 0 && c == 0) {
              ok = mbar_wait_warp_cl(&bars->out_ready[kb], (ready_bits >> kb) & 1, abort_flag, peer_abort, A.status);
              if (!ok) break;
              ready_bits ^= 1u << kb;
              tc_fence_after();
            }
            ok = mbar_wait_warp_cl(&bars->ring_full[s], ph, abort_flag, peer_abort, A.status);
            if (!ok) break;
            const int ksteps = min(128, L.Kpad - kb * 128) >> 5;
            const uint32_t a_lo = desc_lo(a_base + kb * kStageBytes);
            const uint32_t a_tmem = tmem + kActCol + kb * 32;
            const uint32_t b_lo = desc_lo(ring_base + s * kStageBytes);
            if (elect_one()) {
              if (ksteps == 4) {
                if (a_in_tmem) mma2x4_i8_ts(tmem, a_tmem, b_lo, kDescHi, idesc, kb != 0);
                else mma2x4_i8_ss(tmem, a_lo, b_lo, kDescHi, idesc, kb != 0);
              } else {
                const uint64_t adesc = ((uint64_t)kDescHi << 32) | a_lo, bdesc = ((uint64_t)kDescHi << 32) | b_lo;
                for (int ks = 0; ks < ksteps; ++ks) {
                  if (a_in_tmem) mma2_i8_ts(tmem, a_tmem + ks * 8, bdesc + (uint64_t)(ks * 2), idesc, (kb | ks) != 0);
                  else mma2_i8(tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), idesc, (kb | ks) != 0);
                }
              }
              mma_commit_pair(&bars->ring_empty[s], 3);
              if (kb + 1 == L.nkb) {
                mma_commit_pair(&bars->acc_full, 3);
                if (l == 0 && c + 1 == L.nchunk) mma_commit_pair(&bars->a0_empty, 3);
              }
            }
            if (++s == A.n_stages) { s = 0; ph ^= 1; }
          }
        }
      }
    }
    // no MMA of this thread may still be running (in either CTA) when tensor memory is given back
    if (elect_one()) mma_commit_pair(&bars->drain, 1);
    __syncwarp();
    volatile int never = 0;
    mbar_wait_warp(&bars->drain, 0, &never, A.status);
  } else if (warp == 1) {
    // ---------------- relay (odd CTA): "my half of ring stage s has landed" -> even CTA ----------------
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    const uint32_t full0 = mapa_u32(smem_u32(&bars->ring_full[0]), 0);
    for (long long tp = pair_idx; tp < A.n_tile_pairs && ok; tp += n_pairs) {
      for (int i = 0; i < A.stages_per_pair; ++i) {
        ok = mbar_wait_warp(&bars->ring_full[s], ph, abort_flag, A.status);
        if (!ok) break;
        if (lane == 0) mbar_arrive_cluster(full0 + 8u * (uint32_t)s);
        __syncwarp();
        if (++s == A.n_stages) { s = 0; ph ^= 1; }
      }
    }
  } else {
    // ---------------- observation loader / input quantizer (warps 2, 3) ----------------
    const LayerParams p0 = A.params[0];
    const int lw = warp - kLoaderWarp0;
    const int K0 = A.obs_dim;
    const int K0pad128 = A.L[0].nkb * 128;
    const bool vec_ok = ((K0 & 3) == 0) && ((reinterpret_cast<uintptr_t>(A.obs) & 15) == 0);
    const float lo_f = (float)(-128 - p0.z_a), hi_f = (float)(127 - p0.z_a);
    const uint32_t a0_full_leader = mapa_u32(smem_u32(&bars->a0_full), 0);
    uint32_t tp_it = 0;
    bool ok = true;
    for (long long tp = pair_idx; tp < A.n_tile_pairs && ok; tp += n_pairs, ++tp_it) {
      const long long row0 = (2 * tp + rank) * kTileM;
      if (tp_it == 0) {            // shared with the epilogue warps
        load_first_tile(A.obs, A.batch, row0, K0, K0pad128, p0, a0, rs0, lw, kLoaderWarps + kEpiWarps, lane);
        fence_proxy_async();
        mbar_arrive_cluster(mapa_u32(smem_u32(&bars->a0_first), 0));
        continue;
      }
      ok = mbar_wait_warp(&bars->a0_empty, (tp_it - 1) & 1, abort_flag, A.status);
      if (!ok) break;
      const int valid = (int)max(0ll, min((long long)kTileM, A.batch - row0));   // 0: the pair's odd tile does not exist
      int *rowsum0 = rs0 + (tp_it & 1) * kTileM;
      // one lane per observation row, 32 floats at a time, 16-byte shared-memory stores, no shuffles
      for (int rg = lw * 32; rg < kTileM; rg += kLoaderWarps * 32) {
        const int r = rg + lane;
        const float *xrow = A.obs + (valid > 0 ? (row0 + min(r, valid - 1)) * K0 : 0);
        int rsum = 0;
        for (int k0 = 0; k0 < K0pad128; k0 += 32) {
          if (k0 >= K0) continue;     // whole groups of padding columns: written as zeros with the first tile, never changed
          rsum += quantize_obs32(xrow, K0, vec_ok, k0, r < valid, r, p0.inv_s_a, p0.z_a, lo_f, hi_f, a0);
        }
        rowsum0[r] = rsum;
      }
      fence_proxy_async();
      mbar_arrive_cluster(a0_full_leader);
    }
  }
  } else {
    // ---------------- epilogue (warps 4..11) ----------------
    const int ew = warp - kEpiWarp0;
    const int quarter = warp & 3;              // TMEM lanes this warp may touch: 32*quarter .. +31
    const int half = ew >> 2;                  // which 128 columns of a 256-column chunk
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t acc_empty_leader = mapa_u32(smem_u32(&bars->acc_empty), 0);
    const uint32_t out_ready_leader = mapa_u32(smem_u32(&bars->out_ready[0]), 0);
    uint32_t chunk_ctr = 0, tp_it = 0, layer_ctr = 0;
    bool ok = true;
    // column constants of the next layer are fetched one layer ahead, 4 entries per thread
    const int et = threadIdx.x - kEpiWarp0 * 32;                 // 0 .. 255
    auto fetch_cc = [&](int l) -> int4 {
      const Layer &Lc = A.L[l];
      return (4 * et < ((Lc.N + 127) & ~127)) ? __ldg(reinterpret_cast<const int4 *>(Lc.cc) + et) : make_int4(0, 0, 0, 0);
    };
    int4 cc_next = fetch_cc(0);
    if (pair_idx < A.n_tile_pairs) {      // help to load and quantize the first tile's observations
      load_first_tile(A.obs, A.batch, (2 * pair_idx + rank) * kTileM, A.obs_dim, A.L[0].nkb * 128, A.params[0], a0, rs0,
                      kLoaderWarps + ew, kLoaderWarps + kEpiWarps, lane);
      fence_proxy_async();
      mbar_arrive_cluster(mapa_u32(smem_u32(&bars->a0_first), 0));
    }
    for (long long tp = pair_idx; tp < A.n_tile_pairs && ok; tp += n_pairs, ++tp_it) {
      const long long grow = (2 * tp + rank) * kTileM + row;
      const bool row_valid = grow < A.batch;
      int rowsum_in = 0;
      for (int l = 0; l < A.n_layers && ok; ++l, ++layer_ctr) {
        const Layer &L = A.L[l];
        const LayerParams p = A.params[l];
        int4 *cc_buf = cc_smem + (layer_ctr & 1) * (kCcEntries / 4);
        cc_buf[et] = cc_next;
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->cc_ready[layer_ctr & 1]);
        cc_next = fetch_cc(l + 1 == A.n_layers ? 0 : l + 1);
        ok = __all_sync(0xffffffffu, mbar_wait(&bars->cc_ready[layer_ctr & 1], (layer_ctr >> 1) & 1, abort_flag, A.status));
        if (!ok) break;
        const bool last = (l + 1 == A.n_layers);
        const bool dbg = kDbg && (l == A.dbg_layer);
        const bool out_to_tmem = (l & 1) == 0;     // even layers hand their output over in tensor memory
        int rterm = 0;
        const float hi_f = (float)(127 - p.z_out);
        // hidden layers: FMA-pipe requantization to unsigned codes when the output zero-point is -128
        // and the accumulator / multiplier bounds of requant32_u8 hold; otherwise the exact conversions
        const bool out_u8 = L.out_unsigned != 0;
        const bool fast_u8 = out_u8 && (p.M >= 0x1p-15f) && ((long long)L.K * 65025 + p.bias_absmax < (1ll << 29));
        const bool has_cc = !L.a_unsigned || p.bias_absmax != 0;
        const float Ms = p.M * 0x1p-8f, cs = -8388608.0f * Ms;
        int rowsum_out = 0;
        float best_v = 0.0f;
        int best_n = -1;
        const float sigma_row = (last && A.noise != nullptr && row_valid) ? __ldg(A.sigma + grow) : 0.0f;
        for (int c = 0; c < L.nchunk && ok; ++c, ++chunk_ctr) {
          const int rows_c = min(kAccCols, L.Npad - c * kAccCols);
          ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_full, chunk_ctr & 1, abort_flag, A.status));
          if (!ok) break;
          tc_fence_after();
          if (c == 0) {
            if (l == 0) rowsum_in = rs0[(tp_it & 1) * kTileM + row];
            else rowsum_in = rsp[(((l - 1) & 1) * 2 + 0) * kTileM + row] + rsp[(((l - 1) & 1) * 2 + 1) * kTileM + row];
            rterm = -p.z_w * rowsum_in;
          }
          if (!last) {
            // ---- hidden layer: this warp owns columns [64 half, +64) of each 128-column half of the
            // chunk, so that the first half (K block 2c of the next layer) is complete, and released,
            // after half of the arithmetic ----
            // all 128 columns in one go (columns beyond rows_c are allocated and never used), then the
            // accumulator goes back to the MMA issuer before the arithmetic starts
            uint32_t r128[128];
            tmem_ld2x64_wait(tmem + lane_addr + half * 64, tmem + lane_addr + 128 + half * 64, r128);
            const uint32_t (&r)[4][32] = *reinterpret_cast<const uint32_t (*)[4][32]>(&r128);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
            // one copy of the four-slice loop per requantize path (0: FMA pipe, 1: the same plus a column
            // constant, 2: exact conversions), so that the path taken is one contiguous run of code
            auto slices = [&](auto path) {
              constexpr int kPath = decltype(path)::value;
#pragma unroll
              for (int s = 0; s < 4; ++s) {
                const int col0 = (s >> 1) * 128 + half * 64 + (s & 1) * 32;      // column of the chunk
                if (s == 2) {       // K block 2c is written: publish it (after the row sums, if it is the layer's last)
                  if (rows_c <= 128 && c + 1 == L.nchunk) rsp[((l & 1) * 2 + half) * kTileM + row] = rowsum_out;
                  if (out_to_tmem) { tmem_wait_st(); tc_fence_before(); } else fence_proxy_async();
                  __syncwarp();
                  if (lane == 0) mbar_arrive_cluster(out_ready_leader + 8u * (uint32_t)(2 * c));
                  if (rows_c <= 128) return;
                }
                if (col0 >= rows_c) continue;
                const int n0 = c * kAccCols + col0;
                const int4 *cc4 = cc_buf + (n0 >> 2);
                uint32_t packed[8];
                if (kPath == 0) requant32_u8<false>(r[s], cc4, (uint32_t)rterm + 0x4B000000u, Ms, cs, packed);
                else if (kPath == 1) requant32_u8<true>(r[s], cc4, (uint32_t)rterm + 0x4B000000u, Ms, cs, packed);
                else {
                  requant32<0, true>(r[s], cc4, rterm, p.M, hi_f, p.z_out, packed);      // signed codes
                  if (out_u8) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) packed[j] ^= 0x80808080u;
                  }
                }
                if (dbg && row_valid) {
                  for (int j = 0; j < 32; ++j)
                    if (n0 + j < L.N) A.dbg_acc[grow * L.N + n0 + j] = (int)(r[s][j] + (uint32_t)__ldg(L.cc + n0 + j) + (uint32_t)rterm);
                }
                if (n0 + 32 > L.N) {                                 // K padding of the next layer: code 0
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    uint32_t keep = 0;
#pragma unroll
                    for (int e = 0; e < 4; ++e) if (n0 + 4 * j + e < L.N) keep |= 0xffu << (8 * e);
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
                if (dbg && row_valid) {     // the int8 code of an unsigned byte n is n - 128
                  for (int j = 0; j < 32; ++j)
                    if (n0 + j < L.N) A.dbg_act[grow * L.N + n0 + j] = (int8_t)((packed[j >> 2] >> (8 * (j & 3))) ^ (out_u8 ? 0x80u : 0u));
                }
                if (out_to_tmem) {
                  tmem_st8(tmem + lane_addr + kActCol + (n0 >> 2), packed);
                } else {
                  const uint32_t kc = ((uint32_t)n0 & 127) >> 4;     // 16-byte column of the first 16 codes
                  uint8_t *rowp = a_big + ((uint32_t)(n0 >> 7) << 14) + ((uint32_t)row << 7);
                  *reinterpret_cast<uint4 *>(rowp + ((kc ^ ((uint32_t)row & 7)) << 4)) =
                      make_uint4(packed[0], packed[1], packed[2], packed[3]);
                  *reinterpret_cast<uint4 *>(rowp + (((kc + 1) ^ ((uint32_t)row & 7)) << 4)) =
                      make_uint4(packed[4], packed[5], packed[6], packed[7]);
                }
              }
            };
            if (fast_u8) { if (has_cc) slices(PathC<1>{}); else slices(PathC<0>{}); }
            else slices(PathC<2>{});
            // (the row sums are read by the next layer's epilogue, after MMAs that need every K block)
            if (rows_c > 128) {   // K block 2c+1
              if (c + 1 == L.nchunk) rsp[((l & 1) * 2 + half) * kTileM + row] = rowsum_out;
              if (out_to_tmem) { tmem_wait_st(); tc_fence_before(); } else fence_proxy_async();
              __syncwarp();
              if (lane == 0) mbar_arrive_cluster(out_ready_leader + 8u * (uint32_t)(2 * c + 1));
            }
          } else {
            // ---- head: at most 128 columns, done by the half-0 warps ----
            // (the accumulator goes back to the MMA issuer once the last columns are in registers,
            // before the tanh arithmetic)
            // tanh / linear heads: the two warps of a lane quarter take 16 columns each of every 32; a
            // greedy-action head is done by the half-0 warps alone (one running maximum per row)
            const bool split = (A.head != ACTORQ_HEAD_ARGMAX);
            const int n_slices = (split || half == 0) ? (rows_c + 31) / 32 : 0;
            const int sub = split ? half * 16 : 0;
            if (n_slices == 0) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
            }
            // (every column of a slice is computed, without branches, so that the tanh chains of a thread's
            // columns overlap; columns past N never leave: the constants in shared memory are zero-padded)
            auto head_slice = [&](auto width, int col0, bool last_slice) {
              constexpr int kW = decltype(width)::value;          // columns per thread: 16 (split) or 32
              uint32_t r[32];
              tmem_ld32_wait(tmem + lane_addr + col0, r);         // (a split warp uses the first 16 of them)
              if (last_slice) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
              }
              const int n0 = c * kAccCols + col0;
              const int4 *cc4 = cc_buf + (n0 >> 2);
              float y[kW];
#pragma unroll
              for (int j4 = 0; j4 < kW / 4; ++j4) {
                const int4 cc = cc4[j4];
                const int ccv[4] = {cc.x, cc.y, cc.z, cc.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const int acc = (int)(r[4 * j4 + e] + (uint32_t)ccv[e] + (uint32_t)rterm);
                  if (dbg && row_valid && n0 + 4 * j4 + e < L.N) A.dbg_acc[grow * L.N + n0 + 4 * j4 + e] = acc;
                  y[4 * j4 + e] = __fmul_rn(__int2float_rn(acc), p.P);          // Eq. 3 on the accumulator
                }
              }
              if (A.head == ACTORQ_HEAD_ARGMAX) {
#pragma unroll
                for (int j = 0; j < kW; ++j)
                  if (n0 + j < L.N && (y[j] > best_v || best_n < 0)) { best_v = y[j]; best_n = n0 + j; }
              } else if (A.head == ACTORQ_HEAD_TANH) {
#pragma unroll
                for (int j = 0; j < kW; ++j) y[j] = tanhf(y[j]);
                if (A.noise != nullptr && row_valid) {            // actor exploration: y + sigma * eps, kept in [-1, 1]
#pragma unroll
                  for (int j = 0; j < kW; ++j)
                    if (n0 + j < L.N) {
                      const float t = __fadd_rn(y[j], __fmul_rn(sigma_row, __ldg(A.noise + grow * A.out_dim + n0 + j)));
                      y[j] = fminf(fmaxf(t, -1.0f), 1.0f);
                    }
                }
              }
              if (row_valid) {
#pragma unroll
                for (int j = 0; j < kW; ++j)
                  if (n0 + j < L.N) A.out[grow * A.out_dim + n0 + j] = y[j];
              }
            };
            for (int s = 0; s < n_slices; ++s) {
              if (split) head_slice(PathC<16>{}, s * 32 + sub, s + 1 == n_slices);
              else head_slice(PathC<32>{}, s * 32, s + 1 == n_slices);
            }
          }
        }
        if (!ok) break;
        if (last && A.head == ACTORQ_HEAD_ARGMAX && half == 0 && row_valid) A.actions[grow] = best_n;
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

}  // namespace pair

// ---- host side ------------------------------------------------------------------------------

static int round_up_i(int v, int m) { return (v + m - 1) / m * m; }

struct PairPlan { int abig_bytes, a0_bytes, n_stages, smem_bytes; bool ok; };

static PairPlan plan_pair(const actorq_policy *p) {
  PairPlan pl = {0, 0, 0, 0, false};
  if (p->obs_dtype != ACTORQ_OBS_F32) return pl;
  int kmax_hidden = 0;
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerGeom &g = p->layers[l].g;
    if (g.kind != ACTORQ_FC) return pl;
    if (g.K > 1024) return pl;
    const bool last = (l + 1 == p->n_layers);
    if (last ? g.N > 128 : g.N > 1024) return pl;
    if (l >= 2 && (l & 1) == 0 && g.K > kmax_hidden) kmax_hidden = g.K;
  }
  pl.abig_bytes = round_up_i(kmax_hidden, 128) * kTileM;
  pl.a0_bytes = round_up_i(p->layers[0].g.K, 128) * kTileM;
  const int rowsum_bytes = (2 + 4) * kTileM * (int)sizeof(int);
  const int cc_bytes = 2 * pair::kCcEntries * (int)sizeof(int);
  const int fixed = pl.abig_bytes + pl.a0_bytes + (int)sizeof(pair::Barriers) + rowsum_bytes + cc_bytes;
  int stages = (kMaxSmem - fixed) / kStageBytes;
  if (stages > pair::kMaxStages) stages = pair::kMaxStages;
  if (stages < 2) return pl;
  pl.n_stages = stages;
  pl.smem_bytes = fixed + stages * kStageBytes;
  pl.ok = true;
  return pl;
}

bool fused_pair_supported(const actorq_policy *p) { return plan_pair(p).ok; }

int launch_forward_fused_pair(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                              int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st) {
  const PairPlan pl = plan_pair(p);
  if (!pl.ok) return ACTORQ_ERR_UNSUPPORTED;
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
  cfg.blockDim = dim3(pair::kThreads);
  cfg.dynamicSmemBytes = (size_t)pl.smem_bytes;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(pair::fused_mlp_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess ||
        cudaFuncSetAttribute(pair::fused_mlp_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
      return ACTORQ_ERR_CUDA;
    // how many CTA pairs the device can hold at once (shared memory allows one CTA per SM)
    cfg.gridDim = dim3((unsigned)(p->sm_count & ~1));
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, pair::fused_mlp_pair_kernel<false>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
    max_clusters[dev] = n;
    attr_set[dev] = true;
  }
  if (max_clusters[dev] < 1) return ACTORQ_ERR_UNSUPPORTED;

  pair::Args A;
  memset(&A, 0, sizeof(A));
  A.n_layers = p->n_layers;
  int stages_per_pair = 0;
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerDev &L = p->layers[l];
    pair::Layer &F = A.L[l];
    F.img = L.wq_img;
    F.a_unsigned = (l > 0 && p->act[l].z == -128) ? 1 : 0;
    F.out_unsigned = (l + 1 < p->n_layers && p->act[l + 1].z == -128) ? 1 : 0;
    F.cc = F.a_unsigned ? L.bias_q : L.colconst;
    F.K = L.g.K;
    F.N = L.g.N;
    F.Kpad = round_up_i(L.g.K, 32);
    F.Npad = round_up_i(L.g.N, 32);
    F.nkb = (L.g.K + 127) / 128;
    F.nchunk = (F.Npad + pair::kAccCols - 1) / pair::kAccCols;
    stages_per_pair += F.nkb * F.nchunk;
  }
  const long long n_tiles = (batch + kTileM - 1) / kTileM;
  A.params = p->d_params;
  A.obs = (const float *)obs;
  A.batch = batch;
  A.n_tile_pairs = (n_tiles + 1) / 2;
  A.out = out;
  A.actions = actions;
  A.head = p->head;
  if (p->ex_noise != nullptr && p->head == ACTORQ_HEAD_TANH && dbg_layer < 0) {
    A.sigma = p->ex_sigma;
    A.noise = p->ex_noise;
    p->ex_applied = 1;
  }
  A.obs_dim = p->layers[0].g.K;
  A.out_dim = p->layers[p->n_layers - 1].g.N;
  A.n_stages = pl.n_stages;
  A.abig_bytes = pl.abig_bytes;
  A.a0_bytes = pl.a0_bytes;
  A.stages_per_pair = stages_per_pair;
  A.dbg_layer = dbg_layer;
  A.dbg_acc = dbg_acc;
  A.dbg_act = dbg_act;
  A.status = p->d_status;
  // Every CTA pair takes ceil(n_tile_pairs / pairs) tile pairs; launching only as many pairs as that
  // number of rounds needs costs no time and leaves the idle SMs' power to the busy ones' clocks.
  long long pairs = A.n_tile_pairs < max_clusters[dev] ? A.n_tile_pairs : max_clusters[dev];
  const long long rounds = (A.n_tile_pairs + pairs - 1) / pairs;
  pairs = (A.n_tile_pairs + rounds - 1) / rounds;
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  const cudaError_t e = dbg_layer >= 0 ? cudaLaunchKernelEx(&cfg, pair::fused_mlp_pair_kernel<true>, A)
                                       : cudaLaunchKernelEx(&cfg, pair::fused_mlp_pair_kernel<false>, A);
  p->launches++;
  if (e != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_CUDA; }
  return ACTORQ_OK;
}

}  // namespace actorq
