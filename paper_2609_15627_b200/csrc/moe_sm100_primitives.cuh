// Inline-PTX primitives for sm_100a used by the expert-FFN kernels: mbarriers with bounded waits, bulk
// and tensor (TMA) asynchronous copies, tcgen05 tensor-memory allocation, MMA issue, commit and loads.
#pragma once

#include "moe_common.cuh"

namespace moe {

constexpr long long kWaitLimitCycles = 4000000000LL;  // about two seconds of SM clock

MOE_DEVINL uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// ---- mbarrier ---------------------------------------------------------------------------------
MOE_DEVINL void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
MOE_DEVINL void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
MOE_DEVINL void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
MOE_DEVINL void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
MOE_DEVINL bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// The same with a suspend-time hint: the thread may sleep in the instruction, up to about `hint_ns`, until the
// phase completes, instead of spinning - a spinning warp takes issue slots from the warps that share its scheduler.
MOE_DEVINL bool mbar_try_wait_sleepy(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kWaitLimitCycles, records MOE_ERR_TIMEOUT in *status and lets the caller
// go on (the data is then wrong, but every warp keeps taking part in every barrier, so nothing hangs).
// Once the status word is set, every later wait in the grid gives up after a short spin, so that one
// lost signal costs about two seconds in total and not two seconds per wait.
MOE_DEVINL void mbar_wait(uint64_t* bar, uint32_t parity, int* status) {
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait_sleepy(bar, parity, 2000u)) {
    const long long waited = clock64() - t0;
    if (waited > kWaitLimitCycles) {
      if (status != nullptr) atomicExch(status, static_cast<int>(MOE_ERR_TIMEOUT));
      return;
    }
    if (((++spins) & 1023) == 0 && waited > 2000000 && status != nullptr &&
        *reinterpret_cast<volatile int*>(status) != 0)
      return;  // someone already timed out: the results are lost anyway, drain quickly
  }
}

// ---- asynchronous copies ------------------------------------------------------------------------
// contiguous global -> shared, completion counted in bytes on an mbarrier (16-byte aligned, size % 16 == 0)
MOE_DEVINL void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// 2-D tiled tensor-map load into this CTA only; x is the innermost coordinate and x * element size must be a
// multiple of 16 bytes
MOE_DEVINL void tma_load_2d(void* dst, const void* tmap, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(tmap), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
// The same with an L2 cache policy: data that is read once per call (the weight stream) is marked evict-first, so
// that it does not push out what the next call needs again - the kernel's own code, counters, activations.
MOE_DEVINL uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
MOE_DEVINL uint64_t l2_policy_evict_normal() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}
MOE_DEVINL void tma_load_2d_hint(void* dst, const void* tmap, int x, int y, uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(
          smem_u32(dst)),
      "l"(tmap), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
// Output row `row` of the expert FFN: in the caller's y_perm [rows, stride], or - expert-parallel sharding - wherever the
// table says (a row of the buffer of the rank that finishes the row's token, possibly in a peer GPU's memory)
MOE_DEVINL float* y_row(float* y, float* const* row_dst, size_t row, int stride) {
  return row_dst != nullptr ? row_dst[row] : y + row * static_cast<size_t>(stride);
}
// make generic-proxy shared-memory writes visible to the asynchronous proxy (TMA, tcgen05.mma)
MOE_DEVINL void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- tcgen05: tensor memory and MMA ---------------------------------------------------------------
MOE_DEVINL void tmem_alloc(uint32_t* holder_smem, uint32_t ncols) {  // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(holder_smem)), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
MOE_DEVINL void tmem_dealloc(uint32_t taddr, uint32_t ncols) {  // whole warp, the one that allocated
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
MOE_DEVINL void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
MOE_DEVINL void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 operand tile stored as rows of 128 bytes (64
// elements) with the 128-byte swizzle: 8-row groups are 1024 bytes apart; tile base 1024-byte aligned.
MOE_DEVINL uint64_t umma_desc_k_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);  // start address, 16-byte units
  d |= static_cast<uint64_t>(1) << 16;                      // leading byte offset (unused with swizzle)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;              // stride byte offset between 8-row groups
  d |= static_cast<uint64_t>(1) << 46;                      // descriptor version of sm_100
  d |= static_cast<uint64_t>(2) << 61;                      // SWIZZLE_128B
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M x N tile
MOE_DEVINL uint32_t umma_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]^T, issued by one thread
MOE_DEVINL void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
      :
      : "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}
// arrive on an mbarrier when every MMA issued so far by this thread has completed
MOE_DEVINL void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns of tensor memory -> 32 registers per thread (lane = TMEM lane)
MOE_DEVINL void tmem_ld_32x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
MOE_DEVINL void tmem_ld_32x16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
MOE_DEVINL void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- FP4 expansion shared by the FFN kernels -------------------------------------------------------
MOE_DEVINL uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
// bf16x2 of (2^(b-1), 2^(b-1)) for a scale byte b in [0,128]
MOE_DEVINL uint32_t scale_mult(uint32_t b) { return ((b + 126u) << 7) * 0x00010001u; }

// Eight E2M1 codes (one 32-bit word, element i in bits 4i+3:4i) -> four bf16x2 registers holding
// elements (0,4), (1,5), (2,6), (3,7), each multiplied by `m` = bf16x2 of 2^(scale byte - 1).
// A nibble isolated at bit 0 (or 4) and multiplied by 2^6 + 2^12 (or 2^2 + 2^8) lands twice: its
// magnitude bits on bf16 bits 8:6 (value * 2^-126 exactly) and its sign on bit 15; one mask removes the rest.
// k1 = 0x1040 and k2 = 0x0104 are passed in registers the compiler cannot see through (kernel
// parameters), so that each product stays one integer multiply on the FMA pipe instead of being
// rewritten into shift/add pairs on the half-rate integer pipe.
MOE_DEVINL void dequant8(uint32_t wd, uint32_t m, uint32_t k1, uint32_t k2, uint32_t (&p)[4]) {
  constexpr uint32_t kKeep = 0x81C081C0u;
  const uint32_t hi = wd >> 8;
  p[0] = mul_bf16x2(((wd & 0x000F000Fu) * k1) & kKeep, m);
  p[1] = mul_bf16x2(((wd & 0x00F000F0u) * k2) & kKeep, m);
  p[2] = mul_bf16x2(((hi & 0x000F000Fu) * k1) & kKeep, m);
  p[3] = mul_bf16x2(((hi & 0x00F000F0u) * k2) & kKeep, m);
}

}  // namespace moe
