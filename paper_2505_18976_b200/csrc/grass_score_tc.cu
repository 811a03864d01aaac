// grass_score on the 5th-generation tensor cores (tcgen05 + TMEM), fp32-accurate.
//
// scores[i, m] = <train[i, :], test[m, :]> (attribute stage, Section 2.1) is the one dense contraction
// of the path.  fp32 inputs are split exactly into three bf16 pieces, x = hi + mid + lo (8 significant
// bits each, by truncation), and the product is rebuilt from the six partial products whose weight is
// at least 2^-16 of the leading one (hi*hi, hi*mid, mid*hi, mid*mid, hi*lo, lo*hi); what is dropped is
// below 2^-23 of |x||y|, the size of one fp32 rounding.  hi*hi accumulates in one fp32 tile in tensor
// memory and the five correction terms in a second one; the epilogue adds the two.
//
// One CTA owns a 128 x (<=256) output tile: 128 train rows (MMA M) by up to 256 test rows (MMA N).
//   producer warps: read fp32 rows from HBM (the next k tile in registers while the current one is split),
//              split, and write the bf16 pieces into shared memory in the tensor core's K-major layout with
//              the 64-byte swizzle (64-byte rows; conflict-free 16-byte stores); then drain the accumulators;
//   last warp  one elected thread issues tcgen05.mma (M=128, N<=256, K=16) and commits stage-free and
//              accumulator-ready mbarriers.
// Three 72 KB stages of 32 k-values each.  Every mbarrier wait is bounded: if one expires the CTA marks
// its tile with NaN, still frees its tensor memory, and returns.
#include "grass_common.cuh"
#include "tcgen05_util.cuh"

namespace grass {
namespace tc {

constexpr int BM = 128;            // train rows per CTA (MMA M)
constexpr int BN = 256;            // test rows per CTA (MMA N, upper bound)
constexpr int STAGES = 3;
#ifndef GRASS_SCORE_PRODUCERS
#define GRASS_SCORE_PRODUCERS 512
#endif
#ifndef GRASS_SCORE_PREFETCH
#define GRASS_SCORE_PREFETCH 1
#endif
constexpr int PRODUCERS = GRASS_SCORE_PRODUCERS;   // threads of the producer warps
constexpr int PWARPS = PRODUCERS / 32;
constexpr int PF = GRASS_SCORE_PREFETCH;           // k tiles of global loads in flight ahead of the one being split
constexpr int RING = PF + 1;
constexpr int THREADS = PRODUCERS + 32;
constexpr int A_SPLIT_BYTES = BM * BK * 2;   // one bf16 piece of the train tile:  8 KB
constexpr int B_SPLIT_BYTES = BN * BK * 2;   // one bf16 piece of the test tile:  16 KB
constexpr int STAGE_BYTES = 3 * (A_SPLIT_BYTES + B_SPLIT_BYTES);   // 72 KB
constexpr int CHUNKS = BK / 8;     // 16-byte chunks (8 bf16) per row per stage
constexpr int TASKS = (BM + BN) * CHUNKS / PRODUCERS;   // (row, chunk) tasks per producer per stage (3 with 16 producer warps)
constexpr uint32_t TMEM_COLS = 512;   // two fp32 accumulators of BN columns each
__global__ void __launch_bounds__(THREADS, 1)
grass_score_tc_kernel(const float* __restrict__ train, int64_t N, int64_t ld_train, const float* __restrict__ test,
                      int64_t M, int64_t ld_test, int64_t D, float* __restrict__ scores, int64_t ld_s, int vec_ok,
                      int out_vec_ok)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[2 * STAGES + 1];
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t n0 = (int64_t)blockIdx.x * BM;
    const int64_t m0 = (int64_t)blockIdx.y * BN;
    const int64_t m_rows = (M - m0) < BN ? (M - m0) : BN;          // test rows of this tile
    const uint32_t n_mma = (uint32_t)((m_rows + 15) / 16 * 16);    // MMA N (multiple of 16 for M = 128)
    const int64_t ktiles = (D + BK - 1) / BK;

    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]), accum = smem_u32(&bars[2 * STAGES]);
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full0 + 8 * s, PRODUCERS);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accum, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == PWARPS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_slot;
    const uint32_t smem_base = smem_u32(smem);

    if (warp < PWARPS) {
        // ---------------- producers ----------------
        // task q of this thread: flat = tid + q * PRODUCERS -> row = flat / 4 over the 384 rows (train rows
        // first), chunk = flat % 4: four lanes read one row's 128 contiguous bytes, and with the 64-byte
        // swizzle the 16-byte stores of eight consecutive lanes (two rows) fill 128 contiguous bytes
        float raw[RING][TASKS][8];
        auto fetch = [&](int64_t kt, float (&dst)[TASKS][8]) {
            const int64_t d0 = kt * BK;
#pragma unroll
            for (int q = 0; q < TASKS; ++q) {
                const int flat = tid + q * PRODUCERS;
                const int row = flat / CHUNKS, ch = flat % CHUNKS;
                const bool is_a = row < BM;
                const int64_t gr = is_a ? (n0 + row) : (m0 + (row - BM));
                const bool row_ok = is_a ? (gr < N) : (gr < M);
                const float* src = (is_a ? train + gr * ld_train : test + gr * ld_test) + d0 + ch * 8;
                const int64_t d = d0 + ch * 8;
                if (row_ok && vec_ok && d + 7 < D) {
                    const float4 u = __ldg(reinterpret_cast<const float4*>(src));
                    const float4 w = __ldg(reinterpret_cast<const float4*>(src) + 1);
                    dst[q][0] = u.x; dst[q][1] = u.y; dst[q][2] = u.z; dst[q][3] = u.w;
                    dst[q][4] = w.x; dst[q][5] = w.y; dst[q][6] = w.z; dst[q][7] = w.w;
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) dst[q][e] = (row_ok && d + e < D) ? __ldg(src + e) : 0.0f;
                }
            }
        };
        auto stash = [&](int s, const float (&srcv)[TASKS][8]) {
            unsigned char* st = smem + (size_t)s * STAGE_BYTES;
#pragma unroll
            for (int q = 0; q < TASKS; ++q) {
                const int flat = tid + q * PRODUCERS;
                const int row = flat / CHUNKS, ch = flat % CHUNKS;
                const bool is_a = row < BM;
                const int r = is_a ? row : row - BM;
                uint4 hi, mid, lo;
                split8(srcv[q], hi, mid, lo);
                unsigned char* base = is_a ? st : st + 3 * A_SPLIT_BYTES;
                const int piece = is_a ? A_SPLIT_BYTES : B_SPLIT_BYTES;
                const uint32_t off = operand_chunk_offset(r, ch);
                *reinterpret_cast<uint4*>(base + off) = hi;
                *reinterpret_cast<uint4*>(base + piece + off) = mid;
                *reinterpret_cast<uint4*>(base + 2 * piece + off) = lo;
            }
        };
#pragma unroll
        for (int q = 0; q < PF; ++q)
            if (q < ktiles) fetch(q, raw[q]);
        bool ok = true;
        for (int64_t kt0 = 0; kt0 < ktiles && ok; kt0 += RING) {
#pragma unroll
            for (int ph = 0; ph < RING; ++ph) {
                const int64_t kt = kt0 + ph;
                if (kt >= ktiles || !ok) break;
                const int s = (int)(kt % STAGES);
                const uint32_t round = (uint32_t)(kt / STAGES);
                if (kt + PF < ktiles) fetch(kt + PF, raw[(ph + PF) % RING]);
                if (round > 0) ok = mbar_wait(empty0 + 8 * s, (round - 1) & 1) && !abort_flag;
                if (!ok) break;
                stash(s, raw[ph]);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(full0 + 8 * s);
            }
        }
        if (!ok) abort_flag = 1;

        // ---------------- epilogue: drain the accumulator ----------------
        if (ok && ktiles > 0) ok = mbar_wait(accum, 0) && !abort_flag;
        if (!ok) abort_flag = 1;
        ok = __all_sync(0xFFFFFFFFu, ok);   // tensor-memory loads below are warp-collective
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // warp w reads TMEM lanes 32*(w%4) .. +31 (= output rows); the PWARPS/4 warps that share a lane
        // group take every (PWARPS/4)-th 32-column group
        const int lane_grp = warp & 3;
        const int64_t row = n0 + lane_grp * 32 + lane;
        for (uint32_t c0 = (warp >> 2) * 32; c0 < n_mma; c0 += 32 * (PWARPS / 4)) {
            uint32_t v[32];
            if (ok && ktiles > 0) {
                uint32_t w[32];
                tmem_ld32(tmem_d + ((uint32_t)(lane_grp * 32) << 16) + c0, v);
                tmem_ld32(tmem_d + ((uint32_t)(lane_grp * 32) << 16) + BN + c0, w);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) + __uint_as_float(w[e]));
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = (ktiles > 0) ? 0x7FC00000u : 0u;   // NaN marks an aborted tile
            }
            if (row < N) {
                float* dst = scores + row * ld_s + m0 + c0;
                if (out_vec_ok && (int64_t)(c0 + 32) <= m_rows) {
#pragma unroll
                    for (int e = 0; e < 32; e += 4)
                        *reinterpret_cast<uint4*>(dst + e) = make_uint4(v[e], v[e + 1], v[e + 2], v[e + 3]);
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if ((int64_t)(c0 + e) < m_rows) dst[e] = __uint_as_float(v[e]);
                }
            }
        }
    } else if (lane == 0) {
        // ---------------- MMA issuer ----------------
        const uint32_t idesc = make_idesc(BM, n_mma);
        bool ok = true;
        for (int64_t kt = 0; kt < ktiles && ok; ++kt) {
            const int s = (int)(kt % STAGES);
            const uint32_t round = (uint32_t)(kt / STAGES);
            ok = mbar_wait(full0 + 8 * s, round & 1) && !abort_flag;
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_base + s * STAGE_BYTES, b0 = a0 + 3 * A_SPLIT_BYTES;
            // (piece of A, piece of B): 0 = hi, 1 = mid, 2 = lo.  hi*hi goes to the first accumulator, the
            // five correction terms (2^-8 and 2^-16 of it) to the second: the tensor core truncates after
            // every accumulation, so the large sum should see as few of them as possible
            const int pa[6] = {0, 2, 0, 1, 1, 0}, pb[6] = {0, 0, 2, 1, 0, 1};
#pragma unroll
            for (int t = 0; t < 6; ++t) {
#pragma unroll
                for (int ks = 0; ks < BK / 16; ++ks) {
                    const uint64_t ad = make_smem_desc(a0 + pa[t] * A_SPLIT_BYTES + ks * 32);   // 16 k values on
                    const uint64_t bd = make_smem_desc(b0 + pb[t] * B_SPLIT_BYTES + ks * 32);
                    const uint32_t acc_on = (kt > 0 || ks > 0 || t > 1) ? 1u : 0u;
                    umma_bf16(t == 0 ? tmem_d : tmem_d + BN, ad, bd, idesc, acc_on);
                }
            }
            umma_commit(empty0 + 8 * s);   // stage s may be overwritten once these MMAs have read it
        }
        if (!ok) abort_flag = 1;
        if (ok && ktiles > 0) umma_commit(accum);   // accumulator complete
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == PWARPS) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace tc

grass_status launch_score_tc(const float* train, int64_t N, int64_t ld_train, const float* test, int64_t M,
                             int64_t ld_test, int64_t D, float* scores, int64_t ld_s, cudaStream_t st)
{
    const int64_t gx = (N + tc::BM - 1) / tc::BM, gy = (M + tc::BN - 1) / tc::BN;
    if (gx > 0x7FFFFFFFLL || gy > 65535) return GRASS_ERR_UNSUPPORTED;
    const int vec_ok = ((uintptr_t)train % 16 == 0) && ((uintptr_t)test % 16 == 0) && (ld_train % 4 == 0) &&
                       (ld_test % 4 == 0);
    const size_t smem = (size_t)tc::STAGES * tc::STAGE_BYTES + 1024;
    if (cudaFuncSetAttribute(tc::grass_score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
        return GRASS_ERR_CUDA;
    dim3 grid((unsigned)gx, (unsigned)gy);
    const int out_vec_ok = ((uintptr_t)scores % 16 == 0) && (ld_s % 4 == 0);
    tc::grass_score_tc_kernel<<<grid, tc::THREADS, smem, st>>>(train, N, ld_train, test, M, ld_test, D, scores, ld_s,
                                                               vec_ok, out_vec_ok);
    return launch_status();
}

}  // namespace grass
