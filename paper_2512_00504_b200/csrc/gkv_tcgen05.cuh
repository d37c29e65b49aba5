// tcgen05 helpers shared by the tensor-core kernels: shared-memory operand descriptors, the
// instruction descriptor, MMA issue and commit, TMEM loads of 4..32 columns, and a bounded wait that
// gives up early when another role of the CTA has raised its abort flag.
#pragma once

#include "gkv_common.cuh"

namespace gkv {

// K-major operand descriptor: rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart.
// The low word holds the start address in 16-byte units (14 bits; shared memory is < 256 KB, so adding
// a byte offset / 16 never carries out of the field); the high word is the same for every operand.
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t smem_addr) { return ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16); }
__device__ __forceinline__ uint64_t umma_desc(uint32_t lo) {
    constexpr uint32_t hi = 64u | (1u << 14) | (2u << 29);   // stride 1024 B, descriptor version 1, 128-byte swizzle
    return ((uint64_t)hi << 32) | lo;
}
// 16-byte units from the start of an operand tile to its k-step ks (16 elements): d-low / d-high half, then
// 32 bytes per step inside the 128-byte swizzled row.
__device__ __forceinline__ constexpr uint32_t umma_kstep(int ks, int half_bytes) {
    return (uint32_t)(((ks >> 2) * half_bytes + (ks & 3) * 32) >> 4);
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128.
__device__ __forceinline__ uint32_t umma_idesc_bf16_m128(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier gets one arrival once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, float (&v)[N]);
template <>
__device__ __forceinline__ void tmem_ld<8>(uint32_t taddr, float (&v)[8]) {
    uint32_t r[8];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
template <>
__device__ __forceinline__ void tmem_ld<16>(uint32_t taddr, float (&v)[16]) { tmem_ld16(taddr, v); }
template <>
__device__ __forceinline__ void tmem_ld<32>(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Bounded wait that also gives up as soon as another role of the CTA has raised the abort flag.
__device__ __forceinline__ bool tc_wait(uint32_t bar, uint32_t parity, const int* abort_flag) {
    for (uint32_t i = 0; i < kWaitSpins; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*(volatile const int*)abort_flag) return false;
        if (i > 64) __nanosleep(64);
    }
    return false;
}
template <>
__device__ __forceinline__ void tmem_ld<4>(uint32_t taddr, float (&v)[4]) { tmem_ld4(taddr, v); }

}  // namespace gkv
