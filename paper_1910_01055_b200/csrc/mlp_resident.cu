// Fused int8 MLP forward for SMALL policies with the whole quantized policy resident in shared
// memory (sm_100a, tcgen05 cta_group::2) -- paper Section 3.1: actor inference with the quantized
// policy, batched over the observations of many actors; Section 3.2: int8 weights and activations;
// Eq. 1 on the observations, Eq. 3 in the head.
//
// Applies when every layer is one accumulator wide (N <= 256) and at most two 128-byte K blocks
// deep (K <= 256), e.g. the 256-wide D4PG actor networks.  Compared with the streaming kernel in
// mlp_fused_pair.cu:
//   - the int8 weight images of ALL layers are copied into shared memory once per launch (each CTA
//     of a pair holds its half of every layer's rows, 84 KB for 67-256-256-256-21) and stay there:
//     no weight ring and no ring round trips in the per-tile chain;
//   - a full tile of observations (128 rows x obs_dim floats, contiguous in the caller's tensor)
//     arrives as ONE bulk copy into a staging buffer; four loader warps quantize it from shared
//     memory, one lane per row (conflict-free for odd row lengths);
//   - tensor memory holds TWO 256-column accumulators, one per tile slot, and a CTA keeps two tiles
//     in flight: while the epilogue warps requantize layer l of the tile in slot 0 the tensor cores
//     run layer l of the tile in slot 1, and so on alternately.  Each layer being a single chunk, its
//     MMAs have finished reading the layer's input before the epilogue starts, so the next layer's
//     input codes overwrite it in place (one A buffer per slot);
//   - column constants and per-layer parameters of every layer are loaded into shared memory once;
//   - the head: a thread applies Eq. 3, tanh and the exploration noise to 8 columns of its row at a
//     time (8 independent chains) and stores them itself (the outputs are a few KB per tile: staging
//     them in shared memory for coalesced stores cost two rendezvous per tile and was slower).
// Roles per CTA (704 threads): warp 0 bulk-copy producer, warp 1 MMA issuer (even CTA) / relay of
// "my half of the weights has landed" (odd CTA), warps 2-5 observation quantizers, warps 6-21
// epilogue (four per tensor-memory lane quarter, each a quarter of a layer's columns: the requantizer
// is bound by instruction latency with fewer warps per scheduler).  All waits are bounded; a wait that runs out raises ACTORQ_ERR_TIMEOUT and both CTAs'
// abort flags, and both CTAs meet in a cluster barrier before tensor memory is released.
#include <new>
#include "tcgen05.cuh"
#include "explore_rng.cuh"

namespace actorq {

namespace res {

constexpr int kThreads = 704;
constexpr int kLoaderWarp0 = 2;
constexpr int kLoaderWarps = 4;
constexpr int kKParts = kLoaderWarps / 4;   // quantizer warps per 32 rows, each with its own 32-column slices
constexpr int kEpiWarp0 = 6;
constexpr int kEpiWarps = 16;
constexpr int kParts = 4;              // epilogue warps per lane quarter = column parts of a layer
constexpr int kAccCols = 256;

struct Layer {
  const int8_t *img;
  const int *cc;           // per-column integer constant (bias_q for unsigned input codes, else colconst)
  int K, N;
  int Kpad;                // K rounded up to 32 (MMA K step)
  int Npad;                // N rounded up to 32
  int nkb;                 // 128-byte K blocks (1 or 2)
  int half_rows;           // Npad / 2: weight rows each CTA holds
  int w_off;               // byte offset of this layer's weights in the CTA's resident area
  int cc_off;              // offset (ints) of this layer's column constants in shared memory
  int a_unsigned, out_unsigned;
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
  const float *sigma;      // exploration noise (tanh heads) or nullptr
  const float *noise;      // the caller's standard normal draws, or nullptr with noise_seeded: counter-based draws
  int noise_seeded;
  uint32_t seed_lo, seed_hi;
  long long noise_row0;    // absolute row of the call's first observation
  int head;
  float obs_inv_s;         // input quantizer of the observations (host-known: 1 / s_a and z_a of layer 0)
  int obs_z;
  int obs_dim, out_dim;
  int w_bytes;             // resident weights per CTA
  int a_bytes;             // one hidden-activation buffer (per slot)
  int a0_bytes;            // one observation-code buffer (per slot)
  int stage_bytes;         // fp32 staging of one observation tile (0: tiles are read from global memory)
  int cc_ints;
  int dbg_layer;           // -1: none
  int *dbg_acc;
  int8_t *dbg_act;
  int *status;
};

struct __align__(16) Barriers {
  uint64_t w_full[ACTORQ_MAX_LAYERS];
  uint64_t stage_full, stage_empty;
  uint64_t a0_full[2], a0_empty[2];
  uint64_t acc_full[2], a_ready[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Eq. 1 on 32 values of one observation row (one binary32 multiply by 1 / s_a, round half to even,
// clamp) -> 32 codes as two 16-byte pieces of the swizzled A operand; returns the sum of the codes.
// kSmem: the row lies in the shared-memory staging buffer (plain loads), else in global memory.
template <bool kSmem>
__device__ __forceinline__ int quantize_row32(const float *xrow, int K0, bool vec_ok, int k0, bool r_ok, int r,
                                              float inv_s_a, int z_a, float lo_f, float hi_f, uint8_t *a0) {
  float v[32];
  if (vec_ok) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int k = k0 + 4 * i;
      const float4 *src = reinterpret_cast<const float4 *>(xrow + (k < K0 ? k : 0));
      const float4 t = kSmem ? *src : __ldg(src);
      v[4 * i + 0] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = (k0 + i < K0) ? (kSmem ? xrow[k0 + i] : __ldg(xrow + k0 + i)) : 0.0f;
  }
  uint32_t w[8];
  int rsum = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    uint32_t packed = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float t = __fmul_rn(v[4 * i + j], inv_s_a);
      if (t != t) t = 0.0f;                                    // NaN -> real 0
      t = fminf(fmaxf(t, lo_f), hi_f);
      int q = __float_as_int(__fadd_rn(t, 12582912.0f)) - 0x4B400000 + z_a;   // rne at unit spacing
      if (!r_ok || k0 + 4 * i + j >= K0) q = 0;                // rows / columns outside: code 0
      packed |= (uint32_t)(q & 0xff) << (8 * j);
    }
    w[i] = packed;
    rsum = __dp4a((int)packed, 0x01010101, rsum);
  }
  *reinterpret_cast<uint4 *>(a0 + a_offset(r, k0)) = make_uint4(w[0], w[1], w[2], w[3]);
  *reinterpret_cast<uint4 *>(a0 + a_offset(r, k0 + 16)) = make_uint4(w[4], w[5], w[6], w[7]);
  return rsum;
}

template <int V> struct PathC { static constexpr int value = V; };

template <bool kDbg>
__global__ void __launch_bounds__(kThreads, 1)
fused_mlp_resident_kernel(const __grid_constant__ Args A) {
  extern __shared__ __align__(1024) uint8_t smem[];
  if ((smem_u32(smem) & 1023u) != 0) {      // the same in both CTAs of the pair, so both leave
    if (threadIdx.x == 0) atomicMax(A.status, (int)ACTORQ_ERR_CUDA);
    return;
  }
  uint8_t *w_res = smem;
  uint8_t *a_hid = w_res + A.w_bytes;                     // [2 slots][a_bytes]
  uint8_t *a_obs = a_hid + 2 * A.a_bytes;                 // [2 slots][a0_bytes]
  float *stage = reinterpret_cast<float *>(a_obs + 2 * A.a0_bytes);
  Barriers *bars = reinterpret_cast<Barriers *>(reinterpret_cast<uint8_t *>(stage) + A.stage_bytes);
  // partial sums of the observation codes [slot][parity of the slot's tile count][K part][row] (the
  // quantizers may be a whole tile ahead of the epilogue that reads the sums of the slot's current
  // tile) and of each hidden layer's output codes [slot][layer parity][column part][row]; a part
  // covers at most 128 codes, so 16 bits hold its sum
  int16_t *rs0 = reinterpret_cast<int16_t *>(bars + 1);
  int16_t *rsp = rs0 + 8 * kTileM;
  LayerParams *lp = reinterpret_cast<LayerParams *>(rsp + 16 * kTileM);
  int *cc_smem = reinterpret_cast<int *>(lp + ACTORQ_MAX_LAYERS);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const long long pair_idx = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  volatile int *abort_flag = &bars->abort_flag;
  const uint32_t peer_abort = mapa_u32(smem_u32(&bars->abort_flag), rank ^ 1u);
  // tile pairs this CTA pair works through: pair_idx, pair_idx + n_pairs, ...
  const int T = pair_idx < A.n_tile_pairs ? (int)((A.n_tile_pairs - pair_idx + n_pairs - 1) / n_pairs) : 0;

  if (threadIdx.x == 0) {
    for (int l = 0; l < ACTORQ_MAX_LAYERS; ++l) mbar_init(&bars->w_full[l], rank == 0 ? 2 : 1);
    mbar_init(&bars->stage_full, 1);
    mbar_init(&bars->stage_empty, kLoaderWarps);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->a0_full[s], 2 * kLoaderWarps);
      mbar_init(&bars->a0_empty[s], 1);
      mbar_init(&bars->acc_full[s], 1);
      mbar_init(&bars->a_ready[s], 2 * kEpiWarps);
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
  // Launched as a programmatic dependent: everything above may overlap the tail of the previous kernel
  // on the stream (a re-quantization, or the previous forward, whose own dependents are released
  // here); nothing below -- the first read of weights or observations, the first write of outputs --
  // runs before that kernel has completed.
  griddep_launch_dependents();
  griddep_wait();
  const int K0 = A.obs_dim;
  const bool obs_aligned = (reinterpret_cast<uintptr_t>(A.obs) & 15) == 0;

  if (warp == 0) {
    // ---------------- producer: resident weights once, then one bulk copy per full observation tile ----------------
    const bool staging = A.stage_bytes > 0 && obs_aligned;
    uint32_t n_staged = 0;
    int j_next = 0;
    if (staging && T > 0 && (2 * pair_idx + rank + 1) * kTileM <= A.batch) {     // the first tile goes first: the chain starts with it
      if (elect_one()) {
        mbar_expect_tx(&bars->stage_full, (uint32_t)A.stage_bytes);
        bulk_g2s(stage, A.obs + (2 * pair_idx + rank) * kTileM * K0, (uint32_t)A.stage_bytes, &bars->stage_full);
      }
      __syncwarp();
      n_staged = 1;
      j_next = 1;
    }
    if (elect_one()) {
      for (int l = 0; l < A.n_layers; ++l) {
        const Layer &L = A.L[l];
        const int n_first = (int)rank * L.half_rows;
        const int t0 = n_first >> 7, r0 = n_first & 127;
        const int rows_a = min(L.half_rows, 128 - r0), rows_b = L.half_rows - rows_a;
        mbar_expect_tx(&bars->w_full[l], (uint32_t)(L.nkb * L.half_rows * 128));
        for (int kb = 0; kb < L.nkb; ++kb) {
          uint8_t *dst = w_res + L.w_off + kb * L.half_rows * 128;
          bulk_g2s(dst, L.img + (((size_t)t0 * L.nkb + kb) << 14) + ((size_t)r0 << 7), (uint32_t)rows_a * 128, &bars->w_full[l]);
          if (rows_b > 0)
            bulk_g2s(dst + rows_a * 128, L.img + (((size_t)(t0 + 1) * L.nkb + kb) << 14), (uint32_t)rows_b * 128, &bars->w_full[l]);
        }
      }
    }
    __syncwarp();
    bool ok = true;
    if (staging) {
      for (int j = j_next; j < T && ok; ++j) {
        const long long row0 = (2 * (pair_idx + (long long)j * n_pairs) + rank) * kTileM;
        if (row0 + kTileM > A.batch) continue;             // ragged or missing tile: the loaders read global memory
        if (n_staged > 0) {
          ok = mbar_wait_warp(&bars->stage_empty, (n_staged - 1) & 1, abort_flag, A.status);
          if (!ok) break;
        }
        if (elect_one()) {
          mbar_expect_tx(&bars->stage_full, (uint32_t)A.stage_bytes);
          bulk_g2s(stage, A.obs + row0 * K0, (uint32_t)A.stage_bytes, &bars->stage_full);
        }
        __syncwarp();
        ++n_staged;
      }
    }
    if (!ok) {   // leave time for bulk copies still in flight into this CTA's shared memory
      for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
  } else if (warp == 1 && rank == 0) {
    // ---------------- MMA issuer (even CTA): layer by layer, the two tile slots alternating ----------------
    uint32_t a0_use[2] = {0, 0}, ar_cnt[2] = {0, 0};
    bool ok = true;
    for (int j0 = 0; j0 < T && ok; j0 += 2) {
      const int ns = min(2, T - j0);
      for (int l = 0; l < A.n_layers && ok; ++l) {
        const Layer &L = A.L[l];
        const uint32_t idesc = instr_desc_pair(L.Npad, L.a_unsigned != 0);
        if (j0 == 0) {
          ok = mbar_wait_warp_cl(&bars->w_full[l], 0, abort_flag, peer_abort, A.status);
          if (!ok) break;
        }
        for (int s = 0; s < ns && ok; ++s) {
          if (l == 0) {
            ok = mbar_wait_warp_cl(&bars->a0_full[s], a0_use[s] & 1, abort_flag, peer_abort, A.status);
            if (!ok) break;
          }
          if (l > 0 || a0_use[s] > 0) {     // the slot's previous epilogue has read the accumulator / written this layer's input
            ok = mbar_wait_warp_cl(&bars->a_ready[s], ar_cnt[s] & 1, abort_flag, peer_abort, A.status);
            if (!ok) break;
            ++ar_cnt[s];
          }
          tc_fence_after();
          const uint32_t a_base = smem_u32(l == 0 ? a_obs + s * A.a0_bytes : a_hid + s * A.a_bytes);
          const uint32_t b_base = smem_u32(w_res + L.w_off);
          const uint32_t d_tmem = tmem + (uint32_t)s * kAccCols;
          if (elect_one()) {
            for (int kb = 0; kb < L.nkb; ++kb) {
              const int ksteps = min(128, L.Kpad - kb * 128) >> 5;
              const uint32_t a_lo = desc_lo(a_base + kb * kStageBytes);
              const uint32_t b_lo = desc_lo(b_base + kb * L.half_rows * 128);
              if (ksteps == 4) {
                mma2x4_i8_ss(d_tmem, a_lo, b_lo, kDescHi, idesc, kb != 0);
              } else {
                const uint64_t adesc = ((uint64_t)kDescHi << 32) | a_lo, bdesc = ((uint64_t)kDescHi << 32) | b_lo;
                for (int ks = 0; ks < ksteps; ++ks)
                  mma2_i8(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), idesc, (kb | ks) != 0);
              }
            }
            mma_commit_pair(&bars->acc_full[s], 3);
            if (l == 0) mma_commit_pair(&bars->a0_empty[s], 3);
          }
          __syncwarp();
          if (l == 0) ++a0_use[s];
        }
      }
    }
    // no MMA of this thread may still be running (in either CTA) when tensor memory is given back
    if (elect_one()) mma_commit_pair(&bars->drain, 1);
    __syncwarp();
    volatile int never = 0;
    mbar_wait_warp(&bars->drain, 0, &never, A.status);
  } else if (warp == 1) {
    // ---------------- relay (odd CTA): "my half of layer l's weights has landed" -> even CTA ----------------
    const uint32_t full0 = mapa_u32(smem_u32(&bars->w_full[0]), 0);
    for (int l = 0; l < A.n_layers; ++l) {
      if (!mbar_wait_warp(&bars->w_full[l], 0, abort_flag, A.status)) break;
      if (lane == 0) mbar_arrive_cluster(full0 + 8u * (uint32_t)l);
      __syncwarp();
    }
  } else if (warp < kEpiWarp0) {
    // ---------------- observation quantizers (warps 2..5): one lane per row of the tile ----------------
    const float inv_s_a = A.obs_inv_s;
    const int z_a = A.obs_z;
    const int lw = warp - kLoaderWarp0;
    const int r = (lw & 3) * 32 + lane;        // row of the tile
    const int kpart = lw >> 2;                 // this warp's 32-column slices: kpart, kpart + kKParts, ...
    const int K0pad32 = A.L[0].Kpad;
    const bool vec_ok = ((K0 & 3) == 0) && obs_aligned;
    const float lo_f = (float)(-128 - z_a), hi_f = (float)(127 - z_a);
    const uint32_t a0_full_leader = mapa_u32(smem_u32(&bars->a0_full[0]), 0);
    const bool staging = A.stage_bytes > 0 && obs_aligned;
    uint32_t n_staged = 0;
    bool ok = true;
    for (int j = 0; j < T && ok; ++j) {
      const int s = j & 1, use = j >> 1;
      const long long row0 = (2 * (pair_idx + (long long)j * n_pairs) + rank) * kTileM;
      const int valid = (int)max(0ll, min((long long)kTileM, A.batch - row0));    // 0: the pair's odd tile does not exist
      const bool staged = staging && valid == kTileM;
      if (use > 0) {                        // layer 0 of the slot's previous tile has read the codes
        ok = mbar_wait_warp(&bars->a0_empty[s], (use - 1) & 1, abort_flag, A.status);
        if (!ok) break;
      }
      uint8_t *a0 = a_obs + s * A.a0_bytes;
      int rsum = 0;
      if (staged) {
        ok = mbar_wait_warp(&bars->stage_full, n_staged & 1, abort_flag, A.status);
        if (!ok) break;
        const float *xrow = stage + r * K0;
        for (int k0 = 32 * kpart; k0 < K0pad32; k0 += 32 * kKParts)
          rsum += quantize_row32<true>(xrow, K0, vec_ok, k0, true, r, inv_s_a, z_a, lo_f, hi_f, a0);
      } else {
        const float *xrow = A.obs + (valid > 0 ? (row0 + min(r, valid - 1)) * K0 : 0);
        for (int k0 = 32 * kpart; k0 < K0pad32; k0 += 32 * kKParts)
          rsum += quantize_row32<false>(xrow, K0, vec_ok, k0, r < valid, r, inv_s_a, z_a, lo_f, hi_f, a0);
      }
      rs0[((s * 2 + (use & 1)) * 2 + kpart) * kTileM + r] = (int16_t)rsum;
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) {
        if (staged) mbar_arrive(&bars->stage_empty);
        mbar_arrive_cluster(a0_full_leader + 8u * (uint32_t)s);
      }
      if (staged) ++n_staged;
    }
  } else {
    // ---------------- epilogue (warps 6..13) ----------------
    const int ew = warp - kEpiWarp0;
    const int quarter = warp & 3;              // TMEM lanes this warp may touch: 32*quarter .. +31
    const int part = ew >> 2;                  // which quarter of a layer's 32-column slices
    const int row = quarter * 32 + lane;
    const int et = threadIdx.x - kEpiWarp0 * 32;               // 0 .. 255
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t a_ready_leader = mapa_u32(smem_u32(&bars->a_ready[0]), 0);
    // every layer's parameters and column constants into shared memory, once
    if (et < A.n_layers) lp[et] = A.params[et];
    for (int l = 0; l < A.n_layers; ++l) {
      const Layer &Lc = A.L[l];
      for (int i = et; i < Lc.Npad; i += kEpiWarps * 32) cc_smem[Lc.cc_off + i] = (i < Lc.N) ? __ldg(Lc.cc + i) : 0;
    }
    named_bar_sync(1, kEpiWarps * 32);
    uint32_t af_cnt[2] = {0, 0};
    bool ok = true;
    for (int j0 = 0; j0 < T && ok; j0 += 2) {
      const int ns = min(2, T - j0);
      for (int l = 0; l < A.n_layers && ok; ++l) {
        const Layer &L = A.L[l];
        const LayerParams p = lp[l];
        const bool last = (l + 1 == A.n_layers);
        const bool dbg = kDbg && (l == A.dbg_layer);
        const int nsl = L.Npad >> 5;                           // 32-column slices of this layer
        const int4 *cc4 = reinterpret_cast<const int4 *>(cc_smem + L.cc_off);
        for (int s = 0; s < ns && ok; ++s) {
          const long long tile_row0 = (2 * (pair_idx + (long long)(j0 + s) * n_pairs) + rank) * kTileM;
          const long long grow = tile_row0 + row;
          const bool row_valid = grow < A.batch;
          uint8_t *a_out = a_hid + s * A.a_bytes;
          ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_full[s], af_cnt[s] & 1, abort_flag, A.status));
          if (!ok) break;
          ++af_cnt[s];
          tc_fence_after();
          int rs_in;
          if (l == 0) {
            const int16_t *q = rs0 + (s * 2 + ((j0 >> 1) & 1)) * 2 * kTileM + row;
            rs_in = (int)q[0] + (kKParts > 1 ? (int)q[kTileM] : 0);
          } else {
            const int16_t *q = rsp + (s * 2 + ((l - 1) & 1)) * kParts * kTileM + row;
            rs_in = (int)q[0] + (int)q[kTileM] + (int)q[2 * kTileM] + (int)q[3 * kTileM];
          }
          const int rterm = -p.z_w * rs_in;
          const uint32_t acc_addr = tmem + lane_addr + (uint32_t)s * kAccCols;
          if (!last) {
            // ---- hidden layer: requantize this warp's slices and write them, in place of the layer's
            // input, as K blocks of the next layer's A operand ----
            const float hi_f = (float)(127 - p.z_out);
            const bool out_u8 = L.out_unsigned != 0;
            const bool fast_u8 = out_u8 && (p.M >= 0x1p-15f) && ((long long)L.K * 65025 + p.bias_absmax < (1ll << 29));
            const bool has_cc = !L.a_unsigned || p.bias_absmax != 0;
            const float Ms = p.M * 0x1p-8f, cs = -8388608.0f * Ms;
            const int sl0 = (nsl * part) / kParts, sl1 = (nsl * (part + 1)) / kParts;
            int rowsum_out = 0;
            auto slice = [&](auto path, const uint32_t (&r)[32], int sl) {
              constexpr int kPath = decltype(path)::value;
              const int n0 = sl * 32;
              uint32_t packed[8];
              if (kPath == 0) requant32_u8<false>(r, cc4 + (n0 >> 2), (uint32_t)rterm + 0x4B000000u, Ms, cs, packed);
              else if (kPath == 1) requant32_u8<true>(r, cc4 + (n0 >> 2), (uint32_t)rterm + 0x4B000000u, Ms, cs, packed);
              else {
                requant32<0, true>(r, cc4 + (n0 >> 2), rterm, p.M, hi_f, p.z_out, packed);      // signed codes
                if (out_u8) {
#pragma unroll
                  for (int j = 0; j < 8; ++j) packed[j] ^= 0x80808080u;
                }
              }
              if (dbg && row_valid) {
                for (int j = 0; j < 32; ++j)
                  if (n0 + j < L.N) A.dbg_acc[grow * L.N + n0 + j] = (int)(r[j] + (uint32_t)cc_smem[L.cc_off + n0 + j] + (uint32_t)rterm);
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
              const uint32_t kc = ((uint32_t)n0 & 127) >> 4;     // 16-byte column of the first 16 codes
              uint8_t *rowp = a_out + ((uint32_t)(n0 >> 7) << 14) + ((uint32_t)row << 7);
              *reinterpret_cast<uint4 *>(rowp + ((kc ^ ((uint32_t)row & 7)) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
              *reinterpret_cast<uint4 *>(rowp + (((kc + 1) ^ ((uint32_t)row & 7)) << 4)) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
            };
            auto run = [&](auto path) {
              for (int sl = sl0; sl < sl1; ++sl) {
                uint32_t r32[32];
                tmem_ld32_wait(acc_addr + sl * 32, r32);
                slice(path, r32, sl);
              }
            };
            if (fast_u8) { if (has_cc) run(PathC<1>{}); else run(PathC<0>{}); }
            else run(PathC<2>{});
            rsp[((s * 2 + (l & 1)) * kParts + part) * kTileM + row] = (int16_t)rowsum_out;
            tc_fence_before();
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(a_ready_leader + 8u * (uint32_t)s);
          } else {
            // ---- head: Eq. 3 on the accumulator, tanh, exploration noise, stores ----
            const int N = L.N;
            // warp `part` of the quarter dequantizes 8 columns of every 32; a greedy-action head is done by
            // one warp per quarter, which sees whole rows (lowest index among equal maxima)
            const bool greedy = A.head == ACTORQ_HEAD_ARGMAX;
            if (!greedy || part == 0) {
              float best_v = 0.0f;
              int best_n = -1;
              const bool noisy = A.head == ACTORQ_HEAD_TANH && (A.noise != nullptr || A.noise_seeded);
              const float sigma_row = (noisy && row_valid) ? __ldg(A.sigma + grow) : 0.0f;
              // (n0 = 8 nb: the two Philox blocks of a thread's 8 columns are then visibly 2 nb and 2 nb + 1)
              for (int nb = greedy ? 0 : part; nb * 8 < N; nb += greedy ? 1 : kParts) {
                const int n0 = nb * 8;
                uint32_t r[8];
                tmem_ld8_wait(acc_addr + n0, r);
                const int4 c0 = *reinterpret_cast<const int4 *>(cc_smem + L.cc_off + n0);
                const int4 c1 = *reinterpret_cast<const int4 *>(cc_smem + L.cc_off + n0 + 4);
                const int ccv[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
                float y[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  const int acc = (int)(r[j] + (uint32_t)ccv[j] + (uint32_t)rterm);
                  if (dbg && row_valid && n0 + j < N) A.dbg_acc[grow * N + n0 + j] = acc;
                  y[j] = __fmul_rn(__int2float_rn(acc), p.P);                     // Eq. 3
                  if (greedy && n0 + j < N && (y[j] > best_v || best_n < 0)) { best_v = y[j]; best_n = n0 + j; }
                }
                if (A.head == ACTORQ_HEAD_TANH) {
#pragma unroll
                  for (int j = 0; j < 8; ++j) y[j] = tanhf(y[j]);
                  if (noisy && row_valid) {                           // actor exploration: y + sigma * eps, kept in [-1, 1]
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                      if (n0 + j < N) {
                        const float e = A.noise_seeded ? exploration_normal(A.seed_lo, A.seed_hi, A.noise_row0 + grow, nb * 8 + j)
                                                       : __ldg(A.noise + grow * N + n0 + j);
                        y[j] = fminf(fmaxf(__fadd_rn(y[j], __fmul_rn(sigma_row, e)), -1.0f), 1.0f);
                      }
                  }
                }
                if (row_valid) {
#pragma unroll
                  for (int j = 0; j < 8; ++j)
                    if (n0 + j < N) A.out[grow * N + n0 + j] = y[j];
                }
              }
              if (greedy && row_valid) A.actions[grow] = best_n;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(a_ready_leader + 8u * (uint32_t)s);    // the accumulator is free
          }
        }
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

}  // namespace res

// ---- host side ------------------------------------------------------------------------------

static int res_round_up(int v, int m) { return (v + m - 1) / m * m; }

struct ResPlan { int w_bytes, a_bytes, a0_bytes, stage_bytes, cc_ints, smem_bytes; bool ok; };

static ResPlan plan_resident(const actorq_policy *p) {
  ResPlan pl = {0, 0, 0, 0, 0, 0, false};
  if (p->obs_dtype != ACTORQ_OBS_F32) return pl;
  int a_blocks = 1;
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerGeom &g = p->layers[l].g;
    if (g.kind != ACTORQ_FC || g.per_channel) return pl;
    if (g.K > 256 || g.N > 256) return pl;
    const int nkb = (g.K + 127) / 128;
    if (l > 0 && nkb > a_blocks) a_blocks = nkb;
    pl.w_bytes += nkb * (res_round_up(g.N, 32) / 2) * 128;
    pl.cc_ints += res_round_up(g.N, 32);
  }
  pl.a_bytes = a_blocks * kStageBytes;
  pl.a0_bytes = ((p->layers[0].g.K + 127) / 128) * kStageBytes;
  const int misc = (int)sizeof(res::Barriers) + (8 + 16) * kTileM * (int)sizeof(int16_t) +
                   ACTORQ_MAX_LAYERS * (int)sizeof(LayerParams) + pl.cc_ints * (int)sizeof(int) + 64;
  const int fixed = pl.w_bytes + 2 * pl.a_bytes + 2 * pl.a0_bytes + misc;
  const int stage = kTileM * p->layers[0].g.K * (int)sizeof(float);      // 512 * K bytes: a multiple of 16
  if (fixed + stage <= kMaxSmem) pl.stage_bytes = stage;
  else if (fixed > kMaxSmem) return pl;
  pl.smem_bytes = fixed + pl.stage_bytes;
  pl.ok = true;
  return pl;
}

bool fused_resident_supported(const actorq_policy *p) { return plan_resident(p).ok; }

int launch_forward_fused_resident(actorq_policy *p, const void *obs, long long batch, float *out, int *actions,
                                  int dbg_layer, int *dbg_acc, int8_t *dbg_act, cudaStream_t st) {
  const ResPlan pl = plan_resident(p);
  if (!pl.ok) return ACTORQ_ERR_UNSUPPORTED;
  static bool attr_set[64] = {false};
  static int max_clusters[64] = {0};
  const int dev = p->device;
  if (dev < 0 || dev >= 64) return ACTORQ_ERR_UNSUPPORTED;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.blockDim = dim3(res::kThreads);
  cfg.dynamicSmemBytes = (size_t)pl.smem_bytes;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(res::fused_mlp_resident_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess ||
        cudaFuncSetAttribute(res::fused_mlp_resident_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
      return ACTORQ_ERR_CUDA;
    cfg.gridDim = dim3((unsigned)(p->sm_count & ~1));
    cfg.dynamicSmemBytes = (size_t)kMaxSmem;     // one CTA per SM whatever the policy's footprint
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, res::fused_mlp_resident_kernel<false>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
    cfg.dynamicSmemBytes = (size_t)pl.smem_bytes;
    max_clusters[dev] = n;
    attr_set[dev] = true;
  }
  if (max_clusters[dev] < 1) return ACTORQ_ERR_UNSUPPORTED;

  res::Args A;
  memset(&A, 0, sizeof(A));
  A.n_layers = p->n_layers;
  int w_off = 0, cc_off = 0;
  for (int l = 0; l < p->n_layers; ++l) {
    const LayerDev &L = p->layers[l];
    res::Layer &F = A.L[l];
    F.img = L.wq_img;
    F.a_unsigned = (l > 0 && p->act[l].z == -128) ? 1 : 0;
    F.out_unsigned = (l + 1 < p->n_layers && p->act[l + 1].z == -128) ? 1 : 0;
    F.cc = F.a_unsigned ? L.bias_q : L.colconst;
    F.K = L.g.K;
    F.N = L.g.N;
    F.Kpad = res_round_up(L.g.K, 32);
    F.Npad = res_round_up(L.g.N, 32);
    F.nkb = (L.g.K + 127) / 128;
    F.half_rows = F.Npad / 2;
    F.w_off = w_off;
    F.cc_off = cc_off;
    w_off += F.nkb * F.half_rows * 128;
    cc_off += F.Npad;
  }
  const long long n_tiles = (batch + kTileM - 1) / kTileM;
  A.params = p->d_params;
  A.obs = (const float *)obs;
  A.batch = batch;
  A.n_tile_pairs = (n_tiles + 1) / 2;
  A.out = out;
  A.actions = actions;
  A.head = p->head;
  if ((p->ex_noise != nullptr || p->ex_seeded) && p->head == ACTORQ_HEAD_TANH && dbg_layer < 0) {
    A.sigma = p->ex_sigma;
    A.noise = p->ex_noise;
    A.noise_seeded = p->ex_seeded;
    A.seed_lo = (uint32_t)(p->ex_seed & 0xffffffffull);
    A.seed_hi = (uint32_t)(p->ex_seed >> 32);
    A.noise_row0 = p->ex_row0;
    p->ex_applied = 1;
  }
  A.obs_dim = p->layers[0].g.K;
  A.out_dim = p->layers[p->n_layers - 1].g.N;
  A.obs_inv_s = p->act[0].inv_s;
  A.obs_z = p->act[0].z;
  A.w_bytes = pl.w_bytes;
  A.a_bytes = pl.a_bytes;
  A.a0_bytes = pl.a0_bytes;
  A.stage_bytes = pl.stage_bytes;
  A.cc_ints = pl.cc_ints;
  A.dbg_layer = dbg_layer;
  A.dbg_acc = dbg_acc;
  A.dbg_act = dbg_act;
  A.status = p->d_status;
  // every CTA pair takes ceil(n_tile_pairs / pairs) tile pairs; no more pairs than that needs
  long long pairs = A.n_tile_pairs < max_clusters[dev] ? A.n_tile_pairs : max_clusters[dev];
  const long long rounds = (A.n_tile_pairs + pairs - 1) / pairs;
  pairs = (A.n_tile_pairs + rounds - 1) / rounds;
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.numAttrs = 2;
  const cudaError_t e = dbg_layer >= 0 ? cudaLaunchKernelEx(&cfg, res::fused_mlp_resident_kernel<true>, A)
                                       : cudaLaunchKernelEx(&cfg, res::fused_mlp_resident_kernel<false>, A);
  p->launches++;
  if (e != cudaSuccess) { cudaGetLastError(); return ACTORQ_ERR_CUDA; }
  return ACTORQ_OK;
}

}  // namespace actorq
