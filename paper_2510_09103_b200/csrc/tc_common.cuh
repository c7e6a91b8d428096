// Blackwell (sm_100a) building blocks of the tensor-core low-rank path: mbarriers with bounded
// waits, TMA tile loads, tcgen05 MMA / TMEM wrappers and the shared-memory matrix descriptors.
//
// Every operand tile in shared memory is made of boxes of up to 128 rows x 64 bf16 (128 bytes per
// row) written by TMA with the 128-byte swizzle.  Two views of such boxes are used:
//   K-major   rows are the M index, the 64 elements of a row run along K (8-row groups 1024 B
//             apart); the next 64 of K are the next box.
//   MN-major  rows are the K index, the 64 elements of a row run along M (or N).  A wider operand
//             is several boxes side by side, one box size apart; 8-row K groups are 1024 B apart.
// One tcgen05.mma of kind::f16 consumes K = 16: a 32-byte step inside the 128-byte row for a K-major
// operand, two 8-row groups (2048 B) for an MN-major one.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace adapm {
namespace tc {

constexpr int kBoxRows = 128;
constexpr int kBoxCols = 64;                       // bf16 elements: 128 bytes
constexpr int kBoxBytes = kBoxRows * kBoxCols * 2; // 16384
constexpr uint32_t kSpinLimit = 1u << 20;          // bounded waits: about a second of polling in all
constexpr uint32_t kSuspendHintNs = 1000;          // a poll may park the thread this long before it reports failure

// status bits a kernel may set when a bounded wait runs out
enum : int32_t { ST_WAIT_FULL = 1, ST_WAIT_EMPTY = 2, ST_WAIT_TMEM_FULL = 4, ST_WAIT_TMEM_EMPTY = 8, ST_WAIT_DRAIN = 16,
                 ST_WAIT_TEAM = 32 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier ------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("{\n.reg .b64 st;\nmbarrier.arrive.shared::cta.b64 st, [%0];\n}" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("{\n.reg .b64 st;\nmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendHintNs)
      : "memory");
  return ok != 0;
}

// Waits for the phase with the given parity to complete.  Gives up after `limit` polls or as
// soon as another thread of the CTA has given up (*abort != 0); then sets *abort, records `code` in
// the device status word and returns false.  Callers leave their loops on false.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort, int32_t* status,
                                          int32_t code, uint32_t limit = kSpinLimit) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 32) {
      __nanosleep(it > 4096 ? 256 : 32);
      if ((it & 255u) == 0 && *abort) return false;
    }
  }
  *abort = 1;
  atomicOr(status, code);
  return false;
}

// ---- 256-bit global accesses (32-byte aligned addresses) -------------------------------------------
// Eight floats past the L1 (they are used once).
__device__ __forceinline__ void ldcg_f32x8(const float* p, float* v) {
  asm volatile("ld.global.cg.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
               : "l"(p));
}
__device__ __forceinline__ void st_f32x8(float* p, const float* v) {
  asm volatile("st.global.cg.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]),
               "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
               : "memory");
}
__device__ __forceinline__ void st_b32x8(void* p, const uint32_t* v) {
  asm volatile("st.global.cg.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]),
               "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}

// ---- TMA -----------------------------------------------------------------------------------------
// One box at element coordinates (x, y) of a 2-D tensor map; x must be a multiple of 8.
__device__ __forceinline__ void tma_load_box(void* smem_dst, const void* tmap, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(smem_dst)),
      "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

// One box at (x, y, z) of a 3-D tensor map.
__device__ __forceinline__ void tma_load_box3(void* smem_dst, const void* tmap, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
          smem_u32(smem_dst)),
      "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}

// One box from shared memory to element coordinates (x, y) of a 2-D tensor map; elements out of the
// tensor's range are not written.  x * element size must be a multiple of 16 bytes and neither
// coordinate may be negative.  Completion is tracked by the issuing thread's bulk async-groups.
__device__ __forceinline__ void tma_store_box(const void* tmap, int x, int y, const void* smem_src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(tmap), "r"(x),
               "r"(y), "r"(smem_u32(smem_src))
               : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Until at most N of this thread's bulk groups are still reading their shared-memory source.
template <int N>
__device__ __forceinline__ void bulk_wait_group_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
// Until at most N of this thread's bulk groups are incomplete (their writes done).
template <int N>
__device__ __forceinline__ void bulk_wait_group() {
  asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
// Orders this thread's earlier shared-memory writes before later accesses by the async proxy (TMA).
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- tcgen05 -------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
               "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]; issued by one thread.
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier gets one arrival when every MMA this thread issued before has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// 16 consecutive fp32 columns of this thread's TMEM lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, "
      "[%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// The reverse: 16 registers into 16 consecutive columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16};" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
      "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
      "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
      "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- descriptors -----------------------------------------------------------------------------------
// Instruction descriptor of kind::f16 with bf16 operands and fp32 accumulation, M = 128.
__device__ __host__ __forceinline__ uint32_t make_idesc(int n, bool a_mn_major, bool b_mn_major, bool negate_a) {
  uint32_t d = 0;
  d |= 1u << 4;                          // accumulator format: fp32
  d |= 1u << 7;                          // A format: bf16
  d |= 1u << 10;                         // B format: bf16
  d |= (negate_a ? 1u : 0u) << 13;
  d |= (a_mn_major ? 1u : 0u) << 15;
  d |= (b_mn_major ? 1u : 0u) << 16;
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(128 >> 4) << 24;
  return d;
}

// Shared-memory matrix descriptor, 128-byte swizzle (addresses and offsets in 16-byte units).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;                // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                // layout: 128-byte swizzle
  return d;
}
// The same descriptor as two 32-bit halves, so that stepping through K only adds to the low half.
// low: start address and leading byte offset; high: stride byte offset, version, swizzle mode.
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr, uint32_t lbo_bytes) {
  return ((smem_addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__device__ __forceinline__ uint32_t desc_hi() { return (1024u >> 4) | (1u << 14) | (2u << 29); }
__device__ __forceinline__ uint64_t desc_join(uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; }
// K-major operand (8-row groups 1024 B apart); k16 = which 16-wide K step inside the 64-wide box.
__device__ __forceinline__ uint64_t desc_k_major(uint32_t smem_addr, int k16) {
  return desc_join(desc_lo(smem_addr + 32u * (uint32_t)k16, 16), desc_hi());
}
// MN-major operand made of boxes `lbo_bytes` apart; k16 = which 16-row K step inside the box.
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t smem_addr, int k16, uint32_t lbo_bytes) {
  return desc_join(desc_lo(smem_addr + 2048u * (uint32_t)k16, lbo_bytes), desc_hi());
}

// ---- split bf16 --------------------------------------------------------------------------------------
// x ~ hi + lo with both parts bf16 (round to nearest even): the pair carries about 16 significant bits.
// Two values at a time with the packed conversion: returns {hi(x0) | hi(x1) << 16} and the same for lo.
__device__ __forceinline__ uint32_t pack_bf16x2_rn(float x0, float x1) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(x1), "f"(x0));   // first source goes to the upper half
  return d;
}
__device__ __forceinline__ void split_bf16x2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  hi = pack_bf16x2_rn(x0, x1);
  lo = pack_bf16x2_rn(x0 - __uint_as_float(hi << 16), x1 - __uint_as_float(hi & 0xffff0000u));
}
__device__ __forceinline__ void split_bf16(float x, uint16_t& hi, uint16_t& lo) {
  uint32_t h, l;
  split_bf16x2(x, 0.f, h, l);
  hi = (uint16_t)(h & 0xffffu);
  lo = (uint16_t)(l & 0xffffu);
}

}  // namespace tc
}  // namespace adapm
