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

// untiled bulk copy global -> this thread block's shared memory; both addresses 16-byte aligned, `bytes` a multiple
// of 16; completion is counted in bytes on the mbarrier
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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

// two fp32 -> one register of two bf16, round to nearest even, finite inputs stay finite (x0 in the low half)
__device__ __forceinline__ uint32_t pack_bf16x2_rn(float x0, float x1)
{
    uint32_t r;
    asm("cvt.rn.satfinite.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(x1), "f"(x0));
    return r;
}

// eight consecutive fp32 -> three 16-byte chunks of bf16 (hi, mid, lo), x = hi + mid + lo exactly.
// Every piece is the round-to-nearest bf16 of what the pieces before it left over: the two subtractions are
// exact in fp32, the third piece is exact, and hi + mid alone is x rounded to 16-17 significant bits with an
// error of either sign (at most 2^-18 |x|), so that sums of products built from two pieces carry no bias.
__device__ __forceinline__ void split8(const float (&x)[8], uint4& hi, uint4& mid, uint4& lo)
{
    uint32_t h[4], m[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float x0 = x[2 * i], x1 = x[2 * i + 1];
        h[i] = pack_bf16x2_rn(x0, x1);
        const float r0 = x0 - __uint_as_float(h[i] << 16), r1 = x1 - __uint_as_float(h[i] & 0xFFFF0000u);
        m[i] = pack_bf16x2_rn(r0, r1);
        const float s0 = r0 - __uint_as_float(m[i] << 16), s1 = r1 - __uint_as_float(m[i] & 0xFFFF0000u);
        l[i] = pack_bf16x2_rn(s0, s1);
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    mid = make_uint4(m[0], m[1], m[2], m[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

// Partial products of a split fp32 contraction, as (piece of the first operand, piece of the second), 0 = hi,
// 1 = mid, 2 = lo, in the order of their weight: hi*hi; the two terms at 2^-8 of it; mid*mid (2^-16); the two
// hi*lo terms (2^-16).  All six reproduce the fp32 product to 2^-23; the first four to about 2^-17 (unbiased);
// the first three to about 2^-16.  The first goes to an accumulator of its own.
__host__ __device__ constexpr int split_piece_a(int q) { return (q == 2 || q == 3) ? 1 : (q == 5 ? 2 : 0); }
__host__ __device__ constexpr int split_piece_b(int q) { return (q == 1 || q == 3) ? 1 : (q == 4 ? 2 : 0); }
constexpr int kSplitProductsDefault = 6;

}  // namespace tc
}  // namespace grass
