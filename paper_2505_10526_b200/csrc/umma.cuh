// tcgen05 (5th-generation tensor core) wrappers shared by the kernels: fences,
// shared-memory matrix descriptors, single-CTA MMA issue and commit (inline PTX, sm_100a).
#pragma once

#include <stdint.h>

#include "ptx.cuh"

namespace massv {

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte
// swizzle, 8-row groups 1024 bytes apart.  This is the address-independent part.
constexpr uint64_t umma_desc_k_sw128_const() {
    return ((uint64_t)1 << 16)                      // leading byte offset (unused for swizzled K-major)
           | ((uint64_t)(1024 >> 4) << 32)          // stride byte offset between 8-row groups
           | ((uint64_t)1 << 46)                    // descriptor version (sm_100)
           | ((uint64_t)2 << 61);                   // 128-byte swizzle
}

// The descriptor's upper word is the same for every tile; the lower word holds
// the start address, so stepping through a tile is 32-bit arithmetic.
constexpr uint32_t kDescHi = (uint32_t)(umma_desc_k_sw128_const() >> 32);
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t smem_addr) { return ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16); }

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, one CTA.
// ACC = false overwrites D.  Descriptors are passed as (lower word, shared upper word).
template <bool ACC>
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %4};\n\t"
        "mov.b64 db, {%2, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(kDescHi), "r"(ACC ? 1u : 0u)
        : "memory");
}
// Arrive on an mbarrier once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}


// Instruction descriptor of a bf16 x bf16 -> fp32 MMA of shape m x n (x 16); b_mn_major selects a B
// operand whose N index is the contiguous one in shared memory.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int m, int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

}  // namespace massv
