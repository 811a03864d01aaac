// tcgen05 / tensor-memory building blocks shared by the kernels that run their contraction on the
// 5th-generation tensor cores: bounded mbarrier waits, the K-major 64-byte-swizzle shared-memory
// operand layout and its descriptor, MMA issue / commit, tensor-memory loads, and the exact split of
// fp32 into three bf16 pieces.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace grass {
namespace tc {

// Operand tiles hold 32 bf16 k-values per row: 64-byte rows, 8-row groups 512 bytes apart, and the
// 16-byte chunk c of row r stored at chunk position c ^ ((r >> 1) & 3) (the 64-byte swizzle: address
// bits [4,6) xor bits [7,9)).  Tile bases must be 512-byte aligned.
constexpr int BK = 32;                        // k values per shared-memory stage
constexpr uint32_t ROW_BYTES = BK * 2;
constexpr uint32_t SBO = 8 * ROW_BYTES;       // bytes between consecutive 8-row groups (512)
static_assert(ROW_BYTES == 64, "the shared-memory layout is the 64-byte-swizzle K-major one");

// byte offset of the 16-byte chunk `ch` (8 k-values) of row `r` inside an operand tile
__device__ __forceinline__ uint32_t operand_chunk_offset(int r, int ch)
{
    return (uint32_t)((r >> 3) * SBO + (r & 7) * ROW_BYTES + ((ch ^ ((r >> 1) & 3)) << 4));
}

constexpr uint32_t SPIN_LIMIT = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// bounded wait on the phase with the given parity; false if the limit ran out
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < SPIN_LIMIT; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred P;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, P;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

// shared-memory matrix descriptor: K-major, 64-byte swizzle, version 1 (sm_100).  The leading-dimension
// offset is not used by swizzled K-major layouts (set to 16 bytes).  A descriptor that starts 32 bytes
// into the tile addresses k-values 16..31.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)(SBO >> 4) << 32) | (1ull << 46) |
           (4ull << 61);
}

// instruction descriptor: D fp32, A and B bf16, both K-major, M x N
__device__ __forceinline__ uint32_t make_idesc(uint32_t m, uint32_t n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((m >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

// 16 lanes x 32 columns of 32-bit tensor memory, starting at the lane and column in `taddr`, spread over
// the 32 threads of the warp.  Register 4*g + j of thread t holds row (t / 4) + 8 * (j / 2), column
// 8 * g + 2 * (t % 4) + (j % 2)   (g = 0..3: the 16 x 8 fragment of an m16n8 accumulator, repeated).
__device__ __forceinline__ void tmem_ld_16x256b_x4(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

// eight consecutive fp32 -> three 16-byte chunks of bf16 (hi, mid, lo), x = hi + mid + lo exactly
__device__ __forceinline__ void split8(const float (&x)[8], uint4& hi, uint4& mid, uint4& lo)
{
    uint32_t h[8], m[8], l[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t xb = __float_as_uint(x[i]);
        h[i] = xb & 0xFFFF0000u;
        const float r1 = x[i] - __uint_as_float(h[i]);
        m[i] = __float_as_uint(r1) & 0xFFFF0000u;
        const float r2 = r1 - __uint_as_float(m[i]);
        l[i] = __float_as_uint(r2);
    }
    hi = make_uint4(__byte_perm(h[0], h[1], 0x7632), __byte_perm(h[2], h[3], 0x7632), __byte_perm(h[4], h[5], 0x7632),
                    __byte_perm(h[6], h[7], 0x7632));
    mid = make_uint4(__byte_perm(m[0], m[1], 0x7632), __byte_perm(m[2], m[3], 0x7632), __byte_perm(m[4], m[5], 0x7632),
                     __byte_perm(m[6], m[7], 0x7632));
    lo = make_uint4(__byte_perm(l[0], l[1], 0x7632), __byte_perm(l[2], l[3], 0x7632), __byte_perm(l[4], l[5], 0x7632),
                    __byte_perm(l[6], l[7], 0x7632));
}

}  // namespace tc
}  // namespace grass
