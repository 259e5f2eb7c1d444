// Device-side building blocks shared by the tcgen05 kernels: mbarrier / bulk-copy / tcgen05 PTX
// wrappers, bounded waits, UMMA descriptors for K-major 128-byte-swizzled int8 operands, and the
// requantizing epilogue arithmetic.
#pragma once
#include "common.cuh"

namespace actorq {

constexpr int kTileM = 128;            // rows per tile = TMEM lanes
constexpr int kChunkN = 128;           // output columns per accumulator buffer / weight tile
constexpr int kStageBytes = 16384;     // one operand tile: 128 rows x 128 bytes of K
constexpr int kMaxSmem = 232448;       // 227 KB opt-in limit per CTA
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s per wait

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t) :: "memory");     // (not moved across barriers or memory operations)
  return t;
}

// Bounded wait.  Returns false (and raises the abort flag + status word) when the limit runs out
// or another role already aborted.
static __device__ __noinline__ bool mbar_wait_slow(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int *status,
                                                   unsigned long long limit_ns = kWaitLimitNs) {
  unsigned long long t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63) == 0) {
      if (*abort_flag) return false;
      unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > limit_ns || it > (1u << 30)) {
        *abort_flag = 1;
        atomicMax(status, (int)ACTORQ_ERR_TIMEOUT);
        // where it gave up (first reporter only): words 1.. of the status block
        if (atomicCAS(status + 1, 0, 1) == 0) {
          status[2] = (int)blockIdx.x;
          status[3] = (int)(threadIdx.x >> 5);
          status[4] = (int)smem_u32(bar);
          status[5] = (int)parity;
        }
        return false;
      }
    }
  }
}

__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int *status) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status);
}
// one lane polls, the whole warp gets the answer
__device__ __forceinline__ bool mbar_wait_warp(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int *status) {
  // a converged warp reads the same barrier word with one instruction: same answer in every lane
  // (no vote needed on the fast path)
  if (mbar_try_wait(bar, parity)) return true;
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, status) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Programmatic dependent launch: a kernel launched with the programmatic-stream-serialization
// attribute may start while its predecessor in the stream still runs.  griddep_wait() returns once
// the predecessor grid has completed and its memory operations are visible (a no-op when there is
// no such dependency); griddep_launch_dependents() lets the successor start its own set-up early.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// true in exactly one lane of a converged warp
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// K-major operand tile in shared memory, 128-byte swizzle: rows 128 B apart, 8-row groups 1024 B
// apart (stride byte offset), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);        // start address
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset
  d |= (uint64_t)1 << 46;                         // descriptor version
  d |= (uint64_t)2 << 61;                         // SWIZZLE_128B
  return d;
}
// instruction descriptor: D = S32, A = B = signed int8, both K-major, M = 128
__device__ __forceinline__ uint32_t instr_desc(int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// same with the A operand taken from tensor memory (128 lanes = rows, 4 int8 codes per 32-bit column)
__device__ __forceinline__ void mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Four K steps (one full 128-byte K block) in one asm statement: the descriptors differ only in
// their low word (start address advances by 32 bytes = 2 units per step), so they are assembled
// inside the statement from 32-bit pieces and nothing is scheduled between the four MMAs.
__device__ __forceinline__ void mma4_i8_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                           uint32_t idesc, uint32_t acc_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
      "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p0;\n\t"
      "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p1;\n\t"
      "add.u32 al, %1, 4;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p1;\n\t"
      "add.u32 al, %1, 6;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p1;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first) : "memory");
}
__device__ __forceinline__ void mma4_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi,
                                           uint32_t idesc, uint32_t acc_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 db;\n\t.reg .b32 at, bl;\n\t"
      "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], db, %4, p0;\n\t"
      "add.u32 at, %1, 8;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [at], db, %4, p1;\n\t"
      "add.u32 at, %1, 16;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [at], db, %4, p1;\n\t"
      "add.u32 at, %1, 24;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [at], db, %4, p1;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first) : "memory");
}
// low / high words of the K-major 128-byte-swizzle descriptor (see smem_desc)
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr) { return ((saddr & 0x3FFFF) >> 4) | (1u << 16); }
constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);

__device__ __forceinline__ void mma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// tcgen05.ld writes its destination registers asynchronously until tcgen05.wait::ld: the load and
// the wait are one asm statement, so the compiler can never touch the registers in between.
__device__ __forceinline__ void tmem_ld32_wait(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
// 16 columns into the first 16 entries of r
__device__ __forceinline__ void tmem_ld16_wait(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
// one column
__device__ __forceinline__ uint32_t tmem_ld1_wait(uint32_t taddr) {
  uint32_t r;
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r) : "r"(taddr) : "memory");
  return r;
}
// 8 columns
__device__ __forceinline__ void tmem_ld8_wait(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld64_wait(uint32_t taddr, uint32_t (&r)[64]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld128_wait(uint32_t taddr, uint32_t (&r)[128]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x128.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63, %64, %65, %66, %67, %68, %69, %70, %71, %72, %73, %74, %75, %76, %77, %78, %79, %80, %81, %82, %83, %84, %85, %86, %87, %88, %89, %90, %91, %92, %93, %94, %95, %96, %97, %98, %99, %100, %101, %102, %103, %104, %105, %106, %107, %108, %109, %110, %111, %112, %113, %114, %115, %116, %117, %118, %119, %120, %121, %122, %123, %124, %125, %126, %127}, [%128];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]), "=r"(r[64]), "=r"(r[65]), "=r"(r[66]), "=r"(r[67]), "=r"(r[68]), "=r"(r[69]), "=r"(r[70]), "=r"(r[71]), "=r"(r[72]), "=r"(r[73]), "=r"(r[74]), "=r"(r[75]), "=r"(r[76]), "=r"(r[77]), "=r"(r[78]), "=r"(r[79]), "=r"(r[80]), "=r"(r[81]), "=r"(r[82]), "=r"(r[83]), "=r"(r[84]), "=r"(r[85]), "=r"(r[86]), "=r"(r[87]), "=r"(r[88]), "=r"(r[89]), "=r"(r[90]), "=r"(r[91]), "=r"(r[92]), "=r"(r[93]), "=r"(r[94]), "=r"(r[95]), "=r"(r[96]), "=r"(r[97]), "=r"(r[98]), "=r"(r[99]), "=r"(r[100]), "=r"(r[101]), "=r"(r[102]), "=r"(r[103]), "=r"(r[104]), "=r"(r[105]), "=r"(r[106]), "=r"(r[107]), "=r"(r[108]), "=r"(r[109]), "=r"(r[110]), "=r"(r[111]), "=r"(r[112]), "=r"(r[113]), "=r"(r[114]), "=r"(r[115]), "=r"(r[116]), "=r"(r[117]), "=r"(r[118]), "=r"(r[119]), "=r"(r[120]), "=r"(r[121]), "=r"(r[122]), "=r"(r[123]), "=r"(r[124]), "=r"(r[125]), "=r"(r[126]), "=r"(r[127])
      : "r"(taddr) : "memory");
}
// two 64-column loads (r[0..63] from taddr0, r[64..127] from taddr1) behind one wait
__device__ __forceinline__ void tmem_ld2x64_wait(uint32_t taddr0, uint32_t taddr1, uint32_t (&r)[128]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%128];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%64, %65, %66, %67, %68, %69, %70, %71, %72, %73, %74, %75, %76, %77, %78, %79, %80, %81, %82, %83, %84, %85, %86, %87, %88, %89, %90, %91, %92, %93, %94, %95, %96, %97, %98, %99, %100, %101, %102, %103, %104, %105, %106, %107, %108, %109, %110, %111, %112, %113, %114, %115, %116, %117, %118, %119, %120, %121, %122, %123, %124, %125, %126, %127}, [%129];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]), "=r"(r[64]), "=r"(r[65]), "=r"(r[66]), "=r"(r[67]), "=r"(r[68]), "=r"(r[69]), "=r"(r[70]), "=r"(r[71]), "=r"(r[72]), "=r"(r[73]), "=r"(r[74]), "=r"(r[75]), "=r"(r[76]), "=r"(r[77]), "=r"(r[78]), "=r"(r[79]), "=r"(r[80]), "=r"(r[81]), "=r"(r[82]), "=r"(r[83]), "=r"(r[84]), "=r"(r[85]), "=r"(r[86]), "=r"(r[87]), "=r"(r[88]), "=r"(r[89]), "=r"(r[90]), "=r"(r[91]), "=r"(r[92]), "=r"(r[93]), "=r"(r[94]), "=r"(r[95]), "=r"(r[96]), "=r"(r[97]), "=r"(r[98]), "=r"(r[99]), "=r"(r[100]), "=r"(r[101]), "=r"(r[102]), "=r"(r[103]), "=r"(r[104]), "=r"(r[105]), "=r"(r[106]), "=r"(r[107]), "=r"(r[108]), "=r"(r[109]), "=r"(r[110]), "=r"(r[111]), "=r"(r[112]), "=r"(r[113]), "=r"(r[114]), "=r"(r[115]), "=r"(r[116]), "=r"(r[117]), "=r"(r[118]), "=r"(r[119]), "=r"(r[120]), "=r"(r[121]), "=r"(r[122]), "=r"(r[123]), "=r"(r[124]), "=r"(r[125]), "=r"(r[126]), "=r"(r[127])
      : "r"(taddr0), "r"(taddr1) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- CTA pairs (cluster of two, tcgen05 cta_group::2) -----------------------------------------
// One thread of the even CTA issues MMAs that run on both SMs: M = 256 (128 rows from each CTA's
// own A operand), and each CTA supplies half of the B rows from its own shared memory.
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
// Arrive on a barrier that may live in the other CTA of the cluster.  Default semantics (release at
// CTA scope), as for a local arrive: what the waiter consumes has been ordered by the proxy /
// tcgen05 fences executed before the arrive; a cluster-scope release costs over a thousand cycles
// per arrive here.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// waits on a barrier that threads of the other CTA arrive on
__device__ __forceinline__ bool mbar_try_wait_cl(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait for the pair kernel: on expiry both CTAs' abort flags are raised.
static __device__ __noinline__ bool mbar_wait_slow_cl(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                                      uint32_t peer_abort_addr, int *status) {
  unsigned long long t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait_cl(bar, parity)) return true;
    if ((it & 63) == 0) {
      if (*abort_flag) return false;
      unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > kWaitLimitNs || it > (1u << 30)) {
        *abort_flag = 1;
        st_cluster_u32(peer_abort_addr, 1u);
        atomicMax(status, (int)ACTORQ_ERR_TIMEOUT);
        if (atomicCAS(status + 1, 0, 1) == 0) {
          status[2] = (int)blockIdx.x;
          status[3] = (int)(threadIdx.x >> 5);
          status[4] = (int)smem_u32(bar);
          status[5] = (int)parity;
        }
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait_cl(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint32_t peer_abort_addr, int *status) {
  if (mbar_try_wait_cl(bar, parity)) return true;
  return mbar_wait_slow_cl(bar, parity, abort_flag, peer_abort_addr, status);
}
__device__ __forceinline__ bool mbar_wait_warp_cl(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint32_t peer_abort_addr, int *status) {
  if (mbar_try_wait_cl(bar, parity)) return true;
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait_slow_cl(bar, parity, abort_flag, peer_abort_addr, status) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// tensor-memory allocation for a CTA pair: the same warp of BOTH CTAs executes it
__device__ __forceinline__ void tmem_alloc_pair(uint32_t *dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// instruction descriptor for the pair: as instr_desc with M = 256; the A codes are signed int8 or
// (a_unsigned) unsigned 8-bit, B always signed
__device__ __forceinline__ uint32_t instr_desc_pair(int n, bool a_unsigned) {
  return (2u << 4) | ((a_unsigned ? 0u : 1u) << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}
__device__ __forceinline__ void mma2_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma2_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// four K steps of one 128-byte K block (see mma4_i8_ss)
__device__ __forceinline__ void mma2x4_i8_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                             uint32_t idesc, uint32_t acc_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
      "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %4, p0;\n\t"
      "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %4, p1;\n\t"
      "add.u32 al, %1, 4;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %4, p1;\n\t"
      "add.u32 al, %1, 6;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %4, p1;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first) : "memory");
}
__device__ __forceinline__ void mma2x4_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi,
                                             uint32_t idesc, uint32_t acc_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 db;\n\t.reg .b32 at, bl;\n\t"
      "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], [%1], db, %4, p0;\n\t"
      "add.u32 at, %1, 8;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], [at], db, %4, p1;\n\t"
      "add.u32 at, %1, 16;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], [at], db, %4, p1;\n\t"
      "add.u32 at, %1, 24;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 db, {bl, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], [at], db, %4, p1;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first) : "memory");
}
// completion of all MMAs issued so far by this thread -> one arrival on the barrier at this
// shared-memory offset in each CTA named by cta_mask
__device__ __forceinline__ void mma_commit_pair(uint64_t *bar, uint16_t cta_mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(cta_mask) : "memory");
}

// one 32-byte store to global memory (address 32-byte aligned)
__device__ __forceinline__ void st_global_v8(void *p, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t a4, uint32_t a5, uint32_t a6, uint32_t a7) {
  asm volatile("st.global.L1::no_allocate.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"l"(p), "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(a4), "r"(a5), "r"(a6), "r"(a7) : "memory");
}

// A warp holds a tile of 32 rows x W columns of fp32 results, lane = row, bit patterns in v[0..W):
// columns [n0, n0 + W) of out[row0 + lane][.], rows of N floats.  One store per element from its own
// lane would touch 32 cache lines per instruction; instead the tile goes through W * 128 bytes of
// shared memory private to the warp (16-byte pieces, XOR-swizzled so that neither pass has bank
// conflicts) and is written with consecutive lanes on consecutive addresses of a row (32 / W rows
// per instruction).  Rows >= rows_valid and columns >= N are not written.
template <int W>
__device__ __forceinline__ void warp_store_rows(float *__restrict__ out, long long row0, int rows_valid, int N, int n0,
                                                const uint32_t (&v)[32], float *buf, int lane) {
  static_assert(W == 16 || W == 32, "tile width");
  constexpr int kChunks = W / 4, kRowsPerInstr = 32 / W;
  __syncwarp();
#pragma unroll
  for (int j4 = 0; j4 < kChunks; ++j4) {
    const int chunk = j4 ^ ((lane / kRowsPerInstr) & (kChunks - 1));
    *reinterpret_cast<uint4 *>(buf + lane * W + chunk * 4) = make_uint4(v[4 * j4], v[4 * j4 + 1], v[4 * j4 + 2], v[4 * j4 + 3]);
  }
  __syncwarp();
  const int col = lane % W;
  const bool col_ok = n0 + col < N;
#pragma unroll 4
  for (int i = 0; i < W; ++i) {
    const int r = i * kRowsPerInstr + lane / W;
    const int chunk = (col >> 2) ^ ((r / kRowsPerInstr) & (kChunks - 1));
    const float y = buf[r * W + chunk * 4 + (col & 3)];
    if (col_ok && r < rows_valid) out[(row0 + r) * N + n0 + col] = y;
  }
}

// byte offset of activation element (row, k) in an A operand buffer (K blocks of 16 KB)
__device__ __forceinline__ uint32_t a_offset(int row, int k) {
  return ((uint32_t)(k >> 7) << 14) + ((uint32_t)row << 7) + (((((uint32_t)k & 127) >> 4) ^ ((uint32_t)row & 7)) << 4) + ((uint32_t)k & 15);
}

// Input quantizer (Eq. 1 on the observations, one binary32 multiply by 1 / s_a): 32 values of one
// observation row starting at column k0 -> 32 int8 codes written as two 16-byte pieces of the
// swizzled A operand; returns the sum of the codes.  Rows / columns outside the data get code 0.
__device__ __forceinline__ int quantize_obs32(const float *xrow, int K0, bool vec_ok, int k0, bool r_ok, int r,
                                              float inv_s_a, int z_a, float lo_f, float hi_f, uint8_t *a0) {
  float v[32];
  if (vec_ok) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int k = k0 + 4 * i;
      const float4 t = __ldg(reinterpret_cast<const float4 *>(xrow + (k < K0 ? k : 0)));
      v[4 * i + 0] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
    }
  } else {       // rows that are only 4-byte aligned: scalar loads, none for the padding columns
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = (k0 + i < K0) ? __ldg(xrow + k0 + i) : 0.0f;
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
      // |t| <= 255: t + 1.5 * 2^23 rounds half-to-even at unit spacing (no trip through the conversion pipe)
      int q = __float_as_int(__fadd_rn(t, 12582912.0f)) - 0x4B400000 + z_a;
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

// Requantize 32 accumulators of one row to int8 codes, 4 per word:
//   q = clamp(rne((float)acc * M) + z_out, z_out, 127) = rne(clamp((float)acc * M, 0, 127 - z_out)) + z_out
// (rounding is monotone and fixes integers, so the clamp may come first).  Both conversions avoid
// the slow conversion pipe with the 1.5 * 2^23 trick:
//   float -> int: the clamped value lies in [0, 255], so u + 1.5*2^23 rounds half-to-even at unit
//     spacing and its low mantissa bits are rne(u);
//   int -> float (kFast): bits(1.5*2^23) + acc is the float 1.5*2^23 + acc, exactly, while
//     |acc| <= 2^22; beyond that it is still a float of the same sign and magnitude >= 2^22, and the
//     caller only enables kFast when M >= 2^-13 and |acc| < 2^29, so such values clamp to the same
//     end (0 or 127 - z_out) as the exactly converted accumulator would.
// kMode 0: exact cvt.rn.f32.s32 + float clamp (always valid)
// kMode 1: bit-trick int -> float + float clamp (needs M >= 2^-13 and |acc| < 2^29, see above)
// kMode 2: as 1, and the clamp to [0, 255] is done by the saturating 8-bit pack; needs in addition
//          z_out == -128 (the post-ReLU case: the code is the saturated value with its top bit
//          flipped) and M < 2^-8 so that |acc * M| < 2^21 keeps the float -> int trick exact.
__device__ __forceinline__ uint32_t pack_sat_u8(int hi_val, int lo_val, uint32_t upper) {
  uint32_t d;   // d = (upper << 16) | (sat_u8(hi_val) << 8) | sat_u8(lo_val)
  asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(hi_val), "r"(lo_val), "r"(upper));
  return d;
}
// kSharedCC: the column constants are read from shared memory (plain loads) instead of through
// the read-only global path.
template <int kMode, bool kSharedCC = false>
__device__ __forceinline__ void requant32(const uint32_t (&raw)[32], const int4 *__restrict__ cc4, int rterm, float M,
                                          float hi_f, int z_out, uint32_t (&packed)[8]) {
  const float kMagic = 12582912.0f;           // 1.5 * 2^23, bit pattern 0x4B400000
  const int back = (kMode == 2 ? 0 : z_out) - 0x4B400000;
  // acc = raw + colconst[n] - z_w * rowsum_a; in the fast modes the magic bit pattern rides along
  const uint32_t add = (uint32_t)rterm + (kMode != 0 ? 0x4B400000u : 0u);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int4 cc = kSharedCC ? cc4[j] : __ldg(cc4 + j);
    const uint32_t ccv[4] = {(uint32_t)cc.x, (uint32_t)cc.y, (uint32_t)cc.z, (uint32_t)cc.w};
    int q[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t v = raw[4 * j + e] + ccv[e] + add;
      float f;
      if (kMode != 0) f = __fadd_rn(__uint_as_float(v), -kMagic);
      else f = __int2float_rn((int)v);
      float u = __fmul_rn(f, M);
      if (kMode != 2) u = fminf(fmaxf(u, 0.0f), hi_f);
      q[e] = __float_as_int(__fadd_rn(u, kMagic)) + back;
    }
    if (kMode == 2) {
      packed[j] = pack_sat_u8(q[1], q[0], pack_sat_u8(q[3], q[2], 0u)) ^ 0x80808080u;
    } else {
      const uint32_t lo = __byte_perm((uint32_t)q[0], (uint32_t)q[1], 0x0040);
      const uint32_t hi = __byte_perm((uint32_t)q[2], (uint32_t)q[3], 0x0040);
      packed[j] = __byte_perm(lo, hi, 0x5410);
    }
  }
}


// Per-output-channel layers: column n has its own weight zero-point and multiplier, so the row
// term -z_w[n] * rowsum_a is one multiply-add per element and the conversions are the exact ones:
//   acc = raw + colconst[n] - z_w[n] * rowsum_a;  q = rne(clamp((float)acc * M[n], 0, 127 - z_out)) + z_out
__device__ __forceinline__ void requant32_pc(const uint32_t (&raw)[32], const int *__restrict__ cc, const int *__restrict__ zw,
                                             const float *__restrict__ Mn, int rowsum_a, float hi_f, int z_out,
                                             uint32_t (&packed)[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int4 c4 = __ldg(reinterpret_cast<const int4 *>(cc) + j);
    const int4 z4 = __ldg(reinterpret_cast<const int4 *>(zw) + j);
    const float4 m4 = __ldg(reinterpret_cast<const float4 *>(Mn) + j);
    const int ccv[4] = {c4.x, c4.y, c4.z, c4.w}, zv[4] = {z4.x, z4.y, z4.z, z4.w};
    const float mv[4] = {m4.x, m4.y, m4.z, m4.w};
    int q[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int acc = (int)raw[4 * j + e] + ccv[e] - zv[e] * rowsum_a;
      float u = __fmul_rn(__int2float_rn(acc), mv[e]);
      u = fminf(fmaxf(u, 0.0f), hi_f);
      q[e] = __float2int_rn(u) + z_out;
    }
    packed[j] = (uint32_t)(q[0] & 0xff) | ((uint32_t)(q[1] & 0xff) << 8) | ((uint32_t)(q[2] & 0xff) << 16) | ((uint32_t)(q[3] & 0xff) << 24);
  }
}

// Requantize 32 accumulators of one row to UNSIGNED 8-bit codes, 4 per word, for a layer whose
// output zero-point is -128 (post-ReLU range): with u = (float)acc * M rounded to binary32,
//   n = clamp(rne(u), 0, 255) = min(rne(clamp(u, 0, 256)), 255)      (the int8 code is n - 128)
// (rounding is monotone and fixes integers).  Almost everything runs on the FMA pipe:
//   x = bit pattern (2^23 as float) + acc : the float 2^23 + acc exactly for 0 <= acc < 2^23; for
//       acc < 0 some positive float below 2^23, for larger acc some float >= 2^24 (|acc| < 2^29
//       keeps the pattern a positive finite float);
//   s = sat(fma(x, M * 2^-8, -2^23 * M * 2^-8)) : for 0 <= acc < 2^23 the fma rounds the exact
//       acc * M * 2^-8 once, and scaling by a power of two commutes with rounding, so
//       s = clamp(u, 0, 256) / 256; a negative acc gives a negative sum and s = 0; acc >= 2^23
//       gives at least 2^23 * M * 2^-8 >= 1 (M >= 2^-15) and s = 1, as u >= 256 itself would;
//   t = fma(s, 256, 2^23) : 256 s is exact, the sum rounds half-to-even at unit spacing, and the
//       low 16 bits of the pattern are rne(clamp(u, 0, 256)) in [0, 256];
// then two of those per 32-bit word, one 16-bit-lane min with 255, and a byte gather.
// add = (uint32_t)(-z_w * rowsum_a) + 0x4B000000; Ms = M * 2^-8; cs = -2^23 * Ms (both exact).
// kHasCC: a per-column integer constant is added from shared memory.
__device__ __forceinline__ float fma_sat(float a, float b, float c) {
  float d;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint32_t min_u16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("min.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
template <bool kHasCC>
__device__ __forceinline__ void requant32_u8(const uint32_t (&raw)[32], const int4 *__restrict__ cc4, uint32_t add,
                                             float Ms, float cs, uint32_t (&packed)[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    uint32_t ccv[4] = {0u, 0u, 0u, 0u};
    if (kHasCC) {
      const int4 cc = cc4[j];
      ccv[0] = (uint32_t)cc.x; ccv[1] = (uint32_t)cc.y; ccv[2] = (uint32_t)cc.z; ccv[3] = (uint32_t)cc.w;
    }
    uint32_t tb[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t v = raw[4 * j + e] + ccv[e] + add;
      const float sfrac = fma_sat(__uint_as_float(v), Ms, cs);
      tb[e] = __float_as_uint(__fmaf_rn(sfrac, 256.0f, 8388608.0f));
    }
    const uint32_t lo = min_u16x2(__byte_perm(tb[0], tb[1], 0x5410), 0x00FF00FFu);
    const uint32_t hi = min_u16x2(__byte_perm(tb[2], tb[3], 0x5410), 0x00FF00FFu);
    packed[j] = __byte_perm(lo, hi, 0x6420);
  }
}

}  // namespace actorq
