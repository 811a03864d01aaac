// grass_score on the 5th-generation tensor cores (tcgen05 + TMEM), fp32-accurate, CTA pairs, TMA loads.
//
// scores[i, m] = <train[i, :], test[m, :]> (attribute stage, Section 2.1) is the one dense contraction
// of the path.  fp32 inputs are split exactly into three bf16 pieces, x = hi + mid + lo (8 significant
// bits each, by truncation), and the product is rebuilt from the six partial products whose weight is
// at least 2^-16 of the leading one (hi*hi, hi*mid, mid*hi, mid*mid, hi*lo, lo*hi); what is dropped is
// below 2^-23 of |x||y|, the size of one fp32 rounding.  hi*hi accumulates in one fp32 tile in tensor
// memory and the five correction terms in a second one; the epilogue adds the two.
//
// Two CTAs on neighbouring SMs (a cluster of 2) own a 256 x (<=256) output tile and run one
// tcgen05.mma.cta_group::2 (M = 256, N <= 256, K = 16) per product: each CTA stages its own 128 train
// rows and HALF of the test rows, the tensor cores of both SMs read both halves, and each CTA ends up
// with its 128 x N accumulators in its own tensor memory.
//   warp 17    one thread brings the raw fp32 tiles (128 rows x 32 k-values each, train and test) from
//              global memory into a ring of shared-memory slots with TMA (cp.async.bulk.tensor.2d, 128-byte
//              swizzle, each CTA loading only for itself); rows and k-values beyond the matrices arrive as zeros;
//   warps 0-15 producers, in two groups that take alternate k tiles: read a raw slot, split, and write the
//              bf16 pieces into shared memory in the tensor
//              core's K-major layout with the 64-byte swizzle; one lane per warp then arrives on the LEADER
//              CTA's "full" barrier (a remote arrive for the second CTA) and frees the raw slot; afterwards
//              they drain their own CTA's accumulators;
//   warp 16    allocates / frees tensor memory in both CTAs; in the leader CTA one elected thread issues
//              the MMAs and commits, multicast to both CTAs, the stage-free and accumulator-ready barriers.
// Three 48 KB operand stages and two 32 KB raw slots of 32 k-values each.  Every mbarrier wait is bounded:
// if one expires the CTA marks its tile with NaN, still frees its tensor memory, and returns; the cluster
// barriers are reached by every thread of both CTAs unconditionally.
// Long contractions, and outputs with too few tiles to fill the machine, are split over blockIdx.z: every split
// adds its partial products into the zeroed output (see launch_score_tc).
// The TMA path needs 16-byte aligned bases and row strides; other inputs take the plain FMA kernel
// (grass_score.cu).
#include <cuda.h>

#include <algorithm>
#include <cstdlib>

#include "grass_common.cuh"
#include "tcgen05_util.cuh"

namespace grass {
namespace tc {

constexpr int BM = 128;            // train rows per CTA (the pair's MMA M is 256)
constexpr int BN = 256;            // test rows per CTA pair (MMA N, upper bound); each CTA stages half
constexpr int BNH = BN / 2;
constexpr int STAGES = 3;          // bf16 operand stages
constexpr int RING = 2;            // raw fp32 slots filled by TMA
constexpr int PRODUCERS = 512;     // threads of the producer warps
constexpr int PWARPS = PRODUCERS / 32;
constexpr int THREADS = PRODUCERS + 64;   // + the MMA / tensor-memory warp and the TMA warp
constexpr int A_SPLIT_BYTES = BM * BK * 2;    // one bf16 piece of the train tile: 8 KB
constexpr int B_SPLIT_BYTES = BNH * BK * 2;   // one bf16 piece of this CTA's half of the test tile: 8 KB
constexpr int STAGE_BYTES = 3 * (A_SPLIT_BYTES + B_SPLIT_BYTES);   // 48 KB
constexpr int CHUNKS = BK / 8;     // 16-byte chunks (8 bf16) per row per stage
constexpr int GROUPS = 2;          // producer warps work in two groups that take alternate k tiles
constexpr int GROUP_THREADS = PRODUCERS / GROUPS;
constexpr int GROUP_WARPS = PWARPS / GROUPS;
constexpr int TASKS = (BM + BNH) * CHUNKS / GROUP_THREADS;   // (row, chunk) tasks per producer per k tile = 4
// Parity waits are only unambiguous if a waiter never lags a barrier by two phases:
//  - every k tile that uses a given raw slot belongs to the same group (so a group sees all phases of its slots);
//  - a group's previous tile has already waited for an MMA at least as late as the one two rounds back on any stage.
static_assert(RING % GROUPS == 0, "all tiles of a raw slot must belong to one producer group");
static_assert(GROUPS <= STAGES, "operand-stage phases must not be skipped by a producer group");
constexpr uint32_t TMEM_COLS = 512;   // two fp32 accumulators of BN columns each
constexpr int RAW_HALF = BM * BK * 4;            // one raw fp32 tile (128 rows x 32 k-values): 16 KB
constexpr int RAW_BYTES = 2 * RAW_HALF;          // train tile + this CTA's test tile
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + RING * RAW_BYTES;
static_assert(BM == BNH, "both raw tiles use the same TMA box");
static_assert(SMEM_BYTES <= 224 * 1024 && STAGE_BYTES % 1024 == 0 && RAW_HALF % 1024 == 0, "shared memory layout");

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// 2-D tiled TMA load into this CTA's shared memory; x = first k-value (a multiple of 32: 128 bytes), y = first row
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank)
{
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    return ra;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// bounded wait with cluster-scope acquire (the arrivals come from both CTAs)
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < SPIN_LIMIT; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred P;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 P, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, P;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrives on the barrier at this shared-memory offset in both CTAs once all MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask)
                 : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
grass_score_tc_kernel(const __grid_constant__ CUtensorMap map_train, const __grid_constant__ CUtensorMap map_test,
                      int64_t N, int64_t M, int64_t D, int64_t kt_split, float* __restrict__ scores, int64_t ld_s,
                      int out_vec_ok, int nprod)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[2 * STAGES + 1 + 2 * RING];
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();                       // 0 = leader (issues the MMAs)
    const int64_t n0 = (int64_t)blockIdx.x * BM;                   // this CTA's train rows
    const int64_t m0 = (int64_t)blockIdx.y * BN;
    const int64_t m_rows = (M - m0) < BN ? (M - m0) : BN;          // test rows of the pair's tile
    const uint32_t n_mma = (uint32_t)((m_rows + 15) / 16 * 16);    // MMA N (a multiple of 16 for M = 256)
    const int n_half = (int)(n_mma / 2);                           // test rows staged by each CTA
    // blockIdx.z takes k tiles [kt0, kt0 + ktiles); with more than one split the tiles add their partial
    // products into the (zeroed) output
    const int64_t kt0 = (int64_t)blockIdx.z * kt_split;
    const int64_t kt_left = (D + BK - 1) / BK - kt0;
    const int64_t ktiles = kt_left < kt_split ? (kt_left > 0 ? kt_left : 0) : kt_split;
    const bool add_out = gridDim.z > 1;

    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]), accum = smem_u32(&bars[2 * STAGES]);
    const uint32_t rawfull0 = smem_u32(&bars[2 * STAGES + 1]), rawempty0 = rawfull0 + 8 * RING;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full0 + 8 * s, 2 * GROUP_WARPS);   // one arrival per warp of the stage's group in both CTAs
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accum, 1);
        for (int r = 0; r < RING; ++r) {
            mbar_init(rawfull0 + 8 * r, 1);        // the TMA thread's expect_tx arrival + the bytes
            mbar_init(rawempty0 + 8 * r, GROUP_WARPS);   // one arrival per warp of the group that read the slot
        }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == PWARPS) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();            // both CTAs' barriers are initialised before anybody arrives remotely
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_slot;
    const uint32_t smem_base = smem_u32(smem);

    if (warp < PWARPS) {
        // ---------------- producers ----------------
        // The split of one k tile is a latency chain (shared-memory loads, the arithmetic, stores, the proxy
        // fence) about as long as the MMAs of a k tile, so two groups of 8 warps work on alternate k tiles.
        // task q of a thread: flat = (tid % 256) + q * 256 -> row = flat / 4 over the 256 staged rows (128
        // train rows, then this CTA's half of the test rows), chunk = flat % 4 (8 k-values = 32 raw bytes).
        // Raw tiles carry the 128-byte swizzle (16-byte unit u of row r sits at u ^ (r & 7)), operand tiles
        // the 64-byte one: both the 16-byte loads and the 16-byte stores of a quarter warp are conflict-free.
        const unsigned char* raw0 = smem + STAGES * STAGE_BYTES;
        float x[TASKS][8];
        // raw slot -> registers (the slot can be refilled as soon as every warp of the group has done this)
        auto grab = [&](int slot) {
#pragma unroll
            for (int q = 0; q < TASKS; ++q) {
                const int flat = (tid % GROUP_THREADS) + q * GROUP_THREADS;
                const int row = flat / CHUNKS, ch = flat % CHUNKS;
                const bool is_a = row < BM;
                const int r = is_a ? row : row - BM;
                const unsigned char* rt = raw0 + slot * RAW_BYTES + (is_a ? 0 : RAW_HALF) + r * 128;
                const float4 u = *reinterpret_cast<const float4*>(rt + (((2 * ch) ^ (r & 7)) << 4));
                const float4 w = *reinterpret_cast<const float4*>(rt + (((2 * ch + 1) ^ (r & 7)) << 4));
                x[q][0] = u.x; x[q][1] = u.y; x[q][2] = u.z; x[q][3] = u.w;
                x[q][4] = w.x; x[q][5] = w.y; x[q][6] = w.z; x[q][7] = w.w;
            }
        };
        // registers -> the three bf16 pieces of operand stage s
        auto stash = [&](int s) {
            unsigned char* st = smem + (size_t)s * STAGE_BYTES;
#pragma unroll
            for (int q = 0; q < TASKS; ++q) {
                const int flat = (tid % GROUP_THREADS) + q * GROUP_THREADS;
                const int row = flat / CHUNKS, ch = flat % CHUNKS;
                const bool is_a = row < BM;
                const int r = is_a ? row : row - BM;
                uint4 hi, mid, lo;
                split8(x[q], hi, mid, lo);
                unsigned char* base = is_a ? st : st + 3 * A_SPLIT_BYTES;
                const int piece = is_a ? A_SPLIT_BYTES : B_SPLIT_BYTES;
                const uint32_t off = operand_chunk_offset(r, ch);
                *reinterpret_cast<uint4*>(base + off) = hi;
                *reinterpret_cast<uint4*>(base + piece + off) = mid;
                if (nprod > 4) *reinterpret_cast<uint4*>(base + 2 * piece + off) = lo;   // no product reads it otherwise
            }
        };
        const uint32_t leader_full0 = map_to_cta(full0, 0);
        bool ok = true;
        for (int64_t kt = warp / GROUP_WARPS; kt < ktiles; kt += GROUPS) {
            const int s = (int)(kt % STAGES), slot = (int)(kt % RING);
            const uint32_t round = (uint32_t)(kt / STAGES);
            ok = mbar_wait(rawfull0 + 8 * slot, (uint32_t)(kt / RING) & 1) && !abort_flag;      // raw tile landed
            if (!ok) break;
            grab(slot);
            __syncwarp();
            if (lane == 0) mbar_arrive(rawempty0 + 8 * slot);                                     // slot may be refilled
            if (round > 0) ok = mbar_wait(empty0 + 8 * s, (round - 1) & 1) && !abort_flag;         // operand stage free
            if (!ok) break;
            stash(s);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_full0 + 8 * s);
        }
        if (!ok) abort_flag = 1;

        // ---------------- epilogue: drain this CTA's accumulators ----------------
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
                const bool vec = out_vec_ok && (int64_t)(c0 + 32) <= m_rows;
                if (add_out) {
                    if (vec) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + e),
                                         "f"(__uint_as_float(v[e])), "f"(__uint_as_float(v[e + 1])),
                                         "f"(__uint_as_float(v[e + 2])), "f"(__uint_as_float(v[e + 3]))
                                         : "memory");
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if ((int64_t)(c0 + e) < m_rows) atomicAdd(dst + e, __uint_as_float(v[e]));
                    }
                } else if (vec) {
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
    } else if (warp == PWARPS + 1) {
        // ---------------- TMA: raw fp32 tiles into the ring ----------------
        if (lane == 0) {
            const uint32_t raw_u32 = smem_base + STAGES * STAGE_BYTES;
            const int32_t row_a = (int32_t)n0, row_b = (int32_t)(m0 + (int64_t)rank * n_half);
            int64_t issued = 0;
            for (int64_t kt = 0; kt < ktiles; ++kt) {
                const int slot = (int)(kt % RING);
                if (kt >= RING && !(mbar_wait(rawempty0 + 8 * slot, (uint32_t)(kt / RING - 1) & 1) && !abort_flag)) {
                    abort_flag = 1;
                    break;
                }
                mbar_expect_tx(rawfull0 + 8 * slot, RAW_BYTES);
                tma_load_2d(raw_u32 + slot * RAW_BYTES, &map_train, (int32_t)((kt0 + kt) * BK), row_a, rawfull0 + 8 * slot);
                tma_load_2d(raw_u32 + slot * RAW_BYTES + RAW_HALF, &map_test, (int32_t)((kt0 + kt) * BK), row_b, rawfull0 + 8 * slot);
                issued = kt + 1;
            }
            // no copy of this CTA may still be in flight when it leaves (immediate unless the CTA gave up early)
            for (int64_t kt = issued > RING ? issued - RING : 0; kt < issued; ++kt)
                if (!mbar_wait(rawfull0 + 8 * (int)(kt % RING), (uint32_t)(kt / RING) & 1)) abort_flag = 1;
        }
    } else if (lane == 0 && rank == 0) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        const uint32_t idesc = make_idesc(2 * BM, n_mma);
        bool ok = true;
        for (int64_t kt = 0; kt < ktiles && ok; ++kt) {
            const int s = (int)(kt % STAGES);
            const uint32_t round = (uint32_t)(kt / STAGES);
            ok = mbar_wait_cluster(full0 + 8 * s, round & 1) && !abort_flag;
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_base + s * STAGE_BYTES, b0 = a0 + 3 * A_SPLIT_BYTES;
            // hi*hi goes to the first accumulator, the correction terms (2^-8 and 2^-16 of it) to the second:
            // the tensor core truncates after every accumulation, so the large sum should see as few of
            // them as possible
#pragma unroll
            for (int t = 0; t < 6; ++t) {
                if (t >= nprod) break;
#pragma unroll
                for (int ks = 0; ks < BK / 16; ++ks) {
                    const uint64_t ad = make_smem_desc(a0 + split_piece_a(t) * A_SPLIT_BYTES + ks * 32);   // 16 k values on
                    const uint64_t bd = make_smem_desc(b0 + split_piece_b(t) * B_SPLIT_BYTES + ks * 32);
                    const uint32_t acc_on = (kt > 0 || ks > 0 || t > 1) ? 1u : 0u;
                    umma_bf16_pair(t == 0 ? tmem_d : tmem_d + BN, ad, bd, idesc, acc_on);
                }
            }
            umma_commit_pair(empty0 + 8 * s);   // stage s of both CTAs may be overwritten once these MMAs are done
        }
        if (!ok) abort_flag = 1;
        if (ok && ktiles > 0) umma_commit_pair(accum);   // accumulators of both CTAs complete
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();            // nobody leaves while the other CTA may still signal it or read its tiles
    if (warp == PWARPS) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(TMEM_COLS) : "memory");
    }
}


// ---------------------------------------------------------------------------------------------------------
// The same contraction for vectors already stored as bf16 (a cache of compressed gradients at half the size):
// no split is needed, so there are no producer warps at all.  TMA writes the bf16 tiles (128 rows x 64 k-values,
// 128-byte rows, 128-byte swizzle) straight into the K-major operand layout the tensor core reads; per CTA one warp issues the
// loads, one forwards "my tiles have landed" to the leader CTA's barriers, one thread of the leader issues the
// MMAs (one product per 16 k-values), four warps drain the accumulator.
constexpr int H_STAGES = 7;
constexpr int H_BK = 64;                                 // k-values per stage: 128-byte rows, 128-byte swizzle
constexpr int H_ROW_BYTES = H_BK * 2;
constexpr int H_A_BYTES = BM * H_ROW_BYTES;              // this CTA's 128 train rows x 64 k-values of bf16: 16 KB
constexpr int H_B_BYTES = BNH * H_ROW_BYTES;             // this CTA's half of the test rows: 16 KB
constexpr int H_STAGE_BYTES = H_A_BYTES + H_B_BYTES;
constexpr int H_BOX_ROWS = 128;                          // rows per TMA box
constexpr int H_BOXES = BM / H_BOX_ROWS;                 // boxes per operand tile
constexpr int H_EPI_WARPS = 4;
constexpr int H_THREADS = (H_EPI_WARPS + 3) * 32;        // + MMA / tensor-memory warp, TMA warp, forwarding warp
constexpr uint32_t H_TMEM_COLS = 256;                    // one fp32 accumulator of BN columns
static_assert(H_STAGE_BYTES % 1024 == 0 && H_A_BYTES % 1024 == 0, "operand tiles stay 1024-byte aligned");
static_assert(H_STAGES <= 32 && 2 * H_BOXES <= 32 && BM == BNH && (H_BOX_ROWS * H_ROW_BYTES) % 1024 == 0,
              "one stage and one box per lane");
static_assert(H_STAGES * H_STAGE_BYTES <= 224 * 1024, "shared memory");

// shared-memory matrix descriptor for K-major tiles with 128-byte rows and the 128-byte swizzle (8-row groups
// 1,024 bytes apart; 16-byte chunk c of row r stored at chunk c ^ (r & 7)); a descriptor that starts 32 * i bytes
// into the tile addresses k-values 16 i .. 16 i + 15
__device__ __forceinline__ uint64_t make_smem_desc_sw128(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(H_THREADS, 1)
grass_score_bf16_kernel(const __grid_constant__ CUtensorMap map_train, const __grid_constant__ CUtensorMap map_test,
                        int64_t N, int64_t M, int64_t D, int64_t kt_split, float* __restrict__ scores, int64_t ld_s,
                        int out_vec_ok)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[3 * H_STAGES + 1];
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();
    const int64_t n0 = (int64_t)blockIdx.x * BM;
    const int64_t m0 = (int64_t)blockIdx.y * BN;
    const int64_t m_rows = (M - m0) < BN ? (M - m0) : BN;
    const uint32_t n_mma = (uint32_t)((m_rows + 15) / 16 * 16);
    const int n_half = (int)(n_mma / 2);
    const int64_t kt0 = (int64_t)blockIdx.z * kt_split;
    const int64_t kt_left = (D + H_BK - 1) / H_BK - kt0;
    const int64_t ktiles = kt_left < kt_split ? (kt_left > 0 ? kt_left : 0) : kt_split;
    const bool add_out = gridDim.z > 1;

    // landed[s]: this CTA's two tiles of stage s have arrived; full[s] (used in the leader): both CTAs' tiles have;
    // empty[s]: the MMAs that read stage s are done (both CTAs); accum: the accumulators are complete
    const uint32_t landed0 = smem_u32(&bars[0]), full0 = smem_u32(&bars[H_STAGES]), empty0 = smem_u32(&bars[2 * H_STAGES]);
    const uint32_t accum = smem_u32(&bars[3 * H_STAGES]);
    if (tid == 0) {
        for (int s = 0; s < H_STAGES; ++s) {
            mbar_init(landed0 + 8 * s, 1);
            mbar_init(full0 + 8 * s, 2);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accum, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == H_EPI_WARPS) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(H_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_slot;
    const uint32_t smem_base = smem_u32(smem);

    if (warp < H_EPI_WARPS) {
        // ---------------- epilogue: this CTA's 128 rows of the accumulator ----------------
        bool ok = true;
        if (ktiles > 0) ok = mbar_wait(accum, 0) && !abort_flag;
        if (!ok) abort_flag = 1;
        ok = __all_sync(0xFFFFFFFFu, ok);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int64_t row = n0 + warp * 32 + lane;
        for (uint32_t c0 = 0; c0 < n_mma; c0 += 32) {
            uint32_t v[32];
            if (ok && ktiles > 0) {
                tmem_ld32(tmem_d + ((uint32_t)(warp * 32) << 16) + c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = (ktiles > 0) ? 0x7FC00000u : 0u;   // NaN marks an aborted tile
            }
            if (row < N) {
                float* dst = scores + row * ld_s + m0 + c0;
                const bool vec = out_vec_ok && (int64_t)(c0 + 32) <= m_rows;
                if (add_out) {
                    if (vec) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + e),
                                         "f"(__uint_as_float(v[e])), "f"(__uint_as_float(v[e + 1])),
                                         "f"(__uint_as_float(v[e + 2])), "f"(__uint_as_float(v[e + 3]))
                                         : "memory");
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if ((int64_t)(c0 + e) < m_rows) atomicAdd(dst + e, __uint_as_float(v[e]));
                    }
                } else if (vec) {
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
    } else if (warp == H_EPI_WARPS + 1) {
        // ---------------- TMA: bf16 tiles straight into the operand stages ----------------
        // A tile arrives as H_BOXES boxes of H_BOX_ROWS rows, one box per lane.
        const int32_t row_a = (int32_t)n0, row_b = (int32_t)(m0 + (int64_t)rank * n_half);
        int64_t issued = 0;
        bool ok = true;
        for (int64_t kt = 0; kt < ktiles; ++kt) {
            const int s = (int)(kt % H_STAGES);
            const uint32_t round = (uint32_t)(kt / H_STAGES);
            if (lane == 0) {
                if (round > 0) ok = mbar_wait(empty0 + 8 * s, (round - 1) & 1) && !abort_flag;
                if (ok) mbar_expect_tx(landed0 + 8 * s, H_STAGE_BYTES);
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            if (lane < 2 * H_BOXES) {
                const bool is_b = lane >= H_BOXES;
                const int bx = is_b ? lane - H_BOXES : lane;
                const uint32_t dst = smem_base + s * H_STAGE_BYTES + (is_b ? H_A_BYTES : 0) + bx * H_BOX_ROWS * H_ROW_BYTES;
                tma_load_2d(dst, is_b ? &map_test : &map_train, (int32_t)((kt0 + kt) * H_BK),
                            (is_b ? row_b : row_a) + bx * H_BOX_ROWS, landed0 + 8 * s);
            }
            issued = kt + 1;
        }
        if (!ok) abort_flag = 1;
        // no copy of this CTA may still be in flight when it leaves
        if (lane == 0)
            for (int64_t kt = issued > H_STAGES ? issued - H_STAGES : 0; kt < issued; ++kt)
                if (!mbar_wait(landed0 + 8 * (int)(kt % H_STAGES), (uint32_t)(kt / H_STAGES) & 1)) abort_flag = 1;
    } else if (warp == H_EPI_WARPS + 2) {
        // ---------------- forward "landed" to the leader CTA ----------------
        // An arrival on another CTA's barrier takes about a microsecond to return, so one thread forwarding
        // stage after stage would set the pace of the whole kernel.  Lane s looks after stage s instead: the
        // arrivals of several stages are in flight together; every lane polls once per turn of the common loop.
        const uint32_t leader_full0 = map_to_cta(full0, 0);
        int64_t kt = lane;
        bool active = lane < H_STAGES;
        uint32_t spins = 0;
        while (__any_sync(0xFFFFFFFFu, active && kt < ktiles)) {
            if (active && kt < ktiles) {
                uint32_t done;
                asm volatile(
                    "{\n\t.reg .pred P;\n\t"
                    "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
                    "selp.u32 %0, 1, 0, P;\n\t}"
                    : "=r"(done)
                    : "r"(landed0 + 8 * lane), "r"((uint32_t)(kt / H_STAGES) & 1)
                    : "memory");
                if (done) {
                    mbar_arrive_cluster(leader_full0 + 8 * lane);
                    kt += H_STAGES;
                    spins = 0;
                } else if (++spins > SPIN_LIMIT || abort_flag) {
                    abort_flag = 1;
                    active = false;
                }
            }
        }
    } else if (lane == 0 && rank == 0) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        const uint32_t idesc = make_idesc(2 * BM, n_mma);
        bool ok = true;
        for (int64_t kt = 0; kt < ktiles && ok; ++kt) {
            const int s = (int)(kt % H_STAGES);
            ok = mbar_wait_cluster(full0 + 8 * s, (uint32_t)(kt / H_STAGES) & 1) && !abort_flag;
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_base + s * H_STAGE_BYTES, b0 = a0 + H_A_BYTES;
#pragma unroll
            for (int ks = 0; ks < H_BK / 16; ++ks)
                umma_bf16_pair(tmem_d, make_smem_desc_sw128(a0 + ks * 32), make_smem_desc_sw128(b0 + ks * 32), idesc,
                               (kt > 0 || ks > 0) ? 1u : 0u);
            umma_commit_pair(empty0 + 8 * s);
        }
        if (!ok) abort_flag = 1;
        if (ok && ktiles > 0) umma_commit_pair(accum);
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();
    if (warp == H_EPI_WARPS) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(H_TMEM_COLS) : "memory");
    }
}


// ---------------------------------------------------------------------------------------------------------
// bf16 scores with one thread block per 128 x (<= 256) output tile (tcgen05.mma.cta_group::1): for a test set that
// fits one column tile (M <= 256, the usual attribute-stage shape) the pair kernel above gains nothing from sharing
// the test tile between two SMs and pays a remote barrier arrival per stage.  Here every thread block brings in its
// own 128 train rows and ALL test rows of a k tile (the test rows come from L2 after the first block has read
// them), one warp issues the loads, one thread the MMAs, four warps drain the accumulator; all barriers are local.
constexpr int S_STAGES = 4;
constexpr int S_A_BYTES = BM * H_ROW_BYTES;              // 128 train rows x 64 k-values: 16 KB
constexpr int S_B_BYTES = BN * H_ROW_BYTES;              // up to 256 test rows x 64 k-values: 32 KB
constexpr int S_STAGE_BYTES = S_A_BYTES + S_B_BYTES;
constexpr int S_THREADS = (H_EPI_WARPS + 2) * 32;        // + MMA / tensor-memory warp, TMA warp
static_assert(S_STAGES * S_STAGE_BYTES <= 224 * 1024 && S_STAGE_BYTES % 1024 == 0, "shared memory");

__global__ void __launch_bounds__(S_THREADS, 1)
grass_score_bf16_solo_kernel(const __grid_constant__ CUtensorMap map_train, const __grid_constant__ CUtensorMap map_test,
                             int64_t N, int64_t M, int64_t D, int64_t kt_split, float* __restrict__ scores,
                             int64_t ld_s, int out_vec_ok)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[2 * S_STAGES + 1];
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t n0 = (int64_t)blockIdx.x * BM;
    const int64_t m0 = (int64_t)blockIdx.y * BN;
    const int64_t m_rows = (M - m0) < BN ? (M - m0) : BN;
    const uint32_t n_mma = (uint32_t)((m_rows + 15) / 16 * 16);    // MMA N (a multiple of 16 for M = 128)
    const int b_boxes = n_mma > (uint32_t)H_BOX_ROWS ? 2 : 1;      // boxes of 128 test rows per stage
    const int64_t kt0 = (int64_t)blockIdx.z * kt_split;
    const int64_t kt_left = (D + H_BK - 1) / H_BK - kt0;
    const int64_t ktiles = kt_left < kt_split ? (kt_left > 0 ? kt_left : 0) : kt_split;
    const bool add_out = gridDim.z > 1;

    // full[s]: the tiles of stage s have landed; empty[s]: the MMAs that read stage s are done; accum: all MMAs are
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[S_STAGES]), accum = smem_u32(&bars[2 * S_STAGES]);
    if (tid == 0) {
        for (int s = 0; s < S_STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accum, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == H_EPI_WARPS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(H_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_slot;
    const uint32_t smem_base = smem_u32(smem);

    if (warp < H_EPI_WARPS) {
        // ---------------- epilogue: the 128 rows of the accumulator ----------------
        bool ok = true;
        if (ktiles > 0) ok = mbar_wait(accum, 0) && !abort_flag;
        if (!ok) abort_flag = 1;
        ok = __all_sync(0xFFFFFFFFu, ok);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int64_t row = n0 + warp * 32 + lane;
        for (uint32_t c0 = 0; c0 < n_mma; c0 += 32) {
            uint32_t v[32];
            if (ok && ktiles > 0) {
                tmem_ld32(tmem_d + ((uint32_t)(warp * 32) << 16) + c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = (ktiles > 0) ? 0x7FC00000u : 0u;   // NaN marks an aborted tile
            }
            if (row < N) {
                float* dst = scores + row * ld_s + m0 + c0;
                const bool vec = out_vec_ok && (int64_t)(c0 + 32) <= m_rows;
                if (add_out) {
                    if (vec) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + e),
                                         "f"(__uint_as_float(v[e])), "f"(__uint_as_float(v[e + 1])),
                                         "f"(__uint_as_float(v[e + 2])), "f"(__uint_as_float(v[e + 3]))
                                         : "memory");
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if ((int64_t)(c0 + e) < m_rows) atomicAdd(dst + e, __uint_as_float(v[e]));
                    }
                } else if (vec) {
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
    } else if (warp == H_EPI_WARPS + 1) {
        // ---------------- TMA: bf16 tiles straight into the operand stages (one thread) ----------------
        if (lane == 0) {
            const uint32_t stage_tx = (uint32_t)(S_A_BYTES + b_boxes * H_BOX_ROWS * H_ROW_BYTES);
            const int64_t rot = (ktiles > 0 && ktiles <= 128) ? ((int64_t)blockIdx.x * ktiles / gridDim.x) % ktiles : 0;
            int64_t issued = 0;
            bool ok = true;
            for (int64_t kt = 0; kt < ktiles; ++kt) {
                const int s = (int)(kt % S_STAGES);
                const uint32_t round = (uint32_t)(kt / S_STAGES);
                if (round > 0) ok = mbar_wait(empty0 + 8 * s, (round - 1) & 1) && !abort_flag;
                if (!ok) break;
                mbar_expect_tx(full0 + 8 * s, stage_tx);
                const uint32_t dst = smem_base + s * S_STAGE_BYTES;
                // thread blocks walk the k tiles in rotated order (spread evenly over the contraction), so that at
                // any moment they ask L2 for different tiles of the test matrix instead of all for the same one:
                // 65 -> 56 us at 16,384 x 256 x 4,096; for long contractions it measured slower (143 -> 151 us at
                // D = 16,384) and is left out
                const int32_t x = (int32_t)((kt0 + (kt + rot) % ktiles) * H_BK);
                tma_load_2d(dst, &map_train, x, (int32_t)n0, full0 + 8 * s);
                for (int bx = 0; bx < b_boxes; ++bx)
                    tma_load_2d(dst + S_A_BYTES + bx * H_BOX_ROWS * H_ROW_BYTES, &map_test, x,
                                (int32_t)m0 + bx * H_BOX_ROWS, full0 + 8 * s);
                issued = kt + 1;
            }
            if (!ok) abort_flag = 1;
            // no copy of this thread block may still be in flight when it leaves
            for (int64_t kt = issued > S_STAGES ? issued - S_STAGES : 0; kt < issued; ++kt)
                if (!mbar_wait(full0 + 8 * (int)(kt % S_STAGES), (uint32_t)(kt / S_STAGES) & 1)) abort_flag = 1;
        }
    } else if (lane == 0) {
        // ---------------- MMA issuer ----------------
        const uint32_t idesc = make_idesc(BM, n_mma);
        bool ok = true;
        for (int64_t kt = 0; kt < ktiles && ok; ++kt) {
            const int s = (int)(kt % S_STAGES);
            ok = mbar_wait(full0 + 8 * s, (uint32_t)(kt / S_STAGES) & 1) && !abort_flag;
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_base + s * S_STAGE_BYTES, b0 = a0 + S_A_BYTES;
#pragma unroll
            for (int ks = 0; ks < H_BK / 16; ++ks)
                umma_bf16(tmem_d, make_smem_desc_sw128(a0 + ks * 32), make_smem_desc_sw128(b0 + ks * 32), idesc,
                          (kt > 0 || ks > 0) ? 1u : 0u);
            umma_commit(empty0 + 8 * s);
        }
        if (!ok) abort_flag = 1;
        if (ok && ktiles > 0) umma_commit(accum);
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == H_EPI_WARPS) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(H_TMEM_COLS) : "memory");
    }
}

}  // namespace tc

// cuTensorMapEncodeTiled through the runtime's driver entry point (the library does not link libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return (EncodeTiledFn)p;
    }();
    return fn;
}

// rows x D matrix with row stride ld, read in boxes of box_rows rows x 128 bytes with the 128-byte swizzle: 32 fp32
// k-values, or 64 bf16 k-values (then the box is an operand tile as it stands); elements outside the matrix are
// delivered as zeros
static bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t D, int64_t ld, bool bf16 = false,
                     int box_rows = tc::BM)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const size_t esz = bf16 ? 2 : 4;
    const cuuint64_t gdim[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)ld * esz};
    const cuuint32_t box[2] = {(cuuint32_t)(bf16 ? tc::H_BK : tc::BK), (cuuint32_t)box_rows};
    const cuuint32_t estride[2] = {1, 1};
    return enc(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base),
               gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// true if the tensor-core path can take these operands (TMA wants 16-byte aligned bases and row strides)
bool score_tc_supported(const float* train, int64_t ld_train, const float* test, int64_t ld_test, int64_t D)
{
    return D > 0 && ((uintptr_t)train % 16 == 0) && ((uintptr_t)test % 16 == 0) && (ld_train % 4 == 0) &&
           (ld_test % 4 == 0) && encode_tiled_fn() != nullptr;
}

// Split of the contraction over blockIdx.z, for two reasons.  Accuracy: the tensor core truncates the fp32
// accumulator after every MMA, a bias that grows with the number of accumulations, so one accumulator
// never runs over more than 8,192 k-values once D exceeds 16,384 (the partial sums are then added in
// round-to-nearest fp32).  Occupancy: with fewer tile pairs than SM pairs, k is split until the machine
// is about full, in pieces of at least 256 k-values.
static grass_status plan_splits(int64_t D, int64_t pairs, int bk, int64_t* splits_out, int64_t* kt_split_out)
{
    const int64_t ktiles = (D + bk - 1) / bk;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return GRASS_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GRASS_ERR_CUDA;
    int64_t splits = D > 16384 ? (D + 8191) / 8192 : 1;
    if (pairs > 0 && pairs * 2 <= sms / 2) splits = std::max<int64_t>(splits, std::min<int64_t>(sms / 2 / pairs, D / 256));
    splits = tuning(GRASS_TUNE_SCORE_SPLITS, splits);
    splits = std::max<int64_t>(1, std::min<int64_t>(splits, std::min<int64_t>(ktiles, 65535)));
    const int64_t kt_split = (ktiles + splits - 1) / splits;
    *splits_out = (ktiles + kt_split - 1) / kt_split;
    *kt_split_out = kt_split;
    return GRASS_OK;
}

grass_status launch_score_tc(const float* train, int64_t N, int64_t ld_train, const float* test, int64_t M,
                             int64_t ld_test, int64_t D, float* scores, int64_t ld_s, cudaStream_t st)
{
    const int64_t gx = ((N + tc::BM - 1) / tc::BM + 1) / 2 * 2;   // CTA pairs: an even number of row tiles
    const int64_t gy = (M + tc::BN - 1) / tc::BN;
    if (gx > 0x7FFFFFFFLL || gy > 65535 || N > 0x7FFFFFFFLL || M > 0x7FFFFFFFLL || D > 0x7FFFFFFFLL)
        return GRASS_ERR_UNSUPPORTED;
    CUtensorMap map_train, map_test;
    if (!make_map(&map_train, train, N, D, ld_train) || !make_map(&map_test, test, M, D, ld_test)) return GRASS_ERR_CUDA;
    const size_t smem = (size_t)tc::SMEM_BYTES + 1024;
    if (cudaFuncSetAttribute(tc::grass_score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
        return GRASS_ERR_CUDA;
    int64_t splits = 1, kt_split = 1;
    if (plan_splits(D, gx / 2 * gy, tc::BK, &splits, &kt_split) != GRASS_OK) return GRASS_ERR_CUDA;
    if (splits > 1 &&
        cudaMemset2DAsync(scores, (size_t)ld_s * sizeof(float), 0, (size_t)M * sizeof(float), (size_t)N, st) != cudaSuccess)
        return GRASS_ERR_CUDA;
    dim3 grid((unsigned)gx, (unsigned)gy, (unsigned)splits);
    const int out_vec_ok = ((uintptr_t)scores % 16 == 0) && (ld_s % 4 == 0);
    int nprod = (int)tuning(GRASS_TUNE_SPLIT_PRODUCTS, tc::kSplitProductsDefault);
    if (nprod != 3 && nprod != 4) nprod = 6;
    tc::grass_score_tc_kernel<<<grid, tc::THREADS, smem, st>>>(map_train, map_test, N, M, D, kt_split, scores, ld_s,
                                                               out_vec_ok, nprod);
    return launch_status();
}

bool score_bf16_supported(const void* train, int64_t ld_train, const void* test, int64_t ld_test, int64_t D)
{
    return D > 0 && ((uintptr_t)train % 16 == 0) && ((uintptr_t)test % 16 == 0) && (ld_train % 8 == 0) &&
           (ld_test % 8 == 0) && encode_tiled_fn() != nullptr;
}

grass_status launch_score_bf16(const void* train, int64_t N, int64_t ld_train, const void* test, int64_t M,
                               int64_t ld_test, int64_t D, float* scores, int64_t ld_s, cudaStream_t st)
{
    const int64_t gx = ((N + tc::BM - 1) / tc::BM + 1) / 2 * 2;
    const int64_t gy = (M + tc::BN - 1) / tc::BN;
    if (gx > 0x7FFFFFFFLL || gy > 65535 || N > 0x7FFFFFFFLL || M > 0x7FFFFFFFLL || D > 0x7FFFFFFFLL)
        return GRASS_ERR_UNSUPPORTED;
    CUtensorMap map_train, map_test;
    if (!make_map(&map_train, train, N, D, ld_train, true, tc::H_BOX_ROWS) ||
        !make_map(&map_test, test, M, D, ld_test, true, tc::H_BOX_ROWS))
        return GRASS_ERR_CUDA;
    const int out_vec = ((uintptr_t)scores % 16 == 0) && (ld_s % 4 == 0);
    if (gy == 1 && tuning(GRASS_TUNE_SCORE_BF16_SOLO, 1) != 0) {
        // one column tile (M <= 256): one thread block per 128 train rows, no cluster
        const int64_t tiles = (N + tc::BM - 1) / tc::BM;
        const size_t smem1 = (size_t)tc::S_STAGES * tc::S_STAGE_BYTES + 1024;
        if (cudaFuncSetAttribute(tc::grass_score_bf16_solo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem1) != cudaSuccess)
            return GRASS_ERR_CUDA;
        int64_t splits1 = 1, kt_split1 = 1;
        if (plan_splits(D, (tiles + 1) / 2, tc::H_BK, &splits1, &kt_split1) != GRASS_OK) return GRASS_ERR_CUDA;
        if (splits1 > 1 && cudaMemset2DAsync(scores, (size_t)ld_s * sizeof(float), 0, (size_t)M * sizeof(float),
                                             (size_t)N, st) != cudaSuccess)
            return GRASS_ERR_CUDA;
        dim3 grid1((unsigned)tiles, 1, (unsigned)splits1);
        tc::grass_score_bf16_solo_kernel<<<grid1, tc::S_THREADS, smem1, st>>>(map_train, map_test, N, M, D, kt_split1,
                                                                              scores, ld_s, out_vec);
        return launch_status();
    }
    const size_t smem = (size_t)tc::H_STAGES * tc::H_STAGE_BYTES + 1024;
    if (cudaFuncSetAttribute(tc::grass_score_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
        return GRASS_ERR_CUDA;
    int64_t splits = 1, kt_split = 1;
    if (plan_splits(D, gx / 2 * gy, tc::H_BK, &splits, &kt_split) != GRASS_OK) return GRASS_ERR_CUDA;
    if (splits > 1 &&
        cudaMemset2DAsync(scores, (size_t)ld_s * sizeof(float), 0, (size_t)M * sizeof(float), (size_t)N, st) != cudaSuccess)
        return GRASS_ERR_CUDA;
    dim3 grid((unsigned)gx, (unsigned)gy, (unsigned)splits);
    const int out_vec_ok = ((uintptr_t)scores % 16 == 0) && (ld_s % 4 == 0);
    tc::grass_score_bf16_kernel<<<grid, tc::H_THREADS, smem, st>>>(map_train, map_test, N, M, D, kt_split, scores, ld_s,
                                                                   out_vec_ok);
    return launch_status();
}

}  // namespace grass
