// FactGraSS (Section 3.3.2) for launches of about one wave: one thread-block cluster per (layer, sample).
//
// The streaming kernel (factgrass.cu) splits a sample's token sum over independent thread blocks that each
// project their partial block and add the projection into a zeroed output row.  With few work items that costs a
// zero-fill launch, global reductions and one full set of hashes per token chunk, none of it overlapped with loads.
// Here the NC thread blocks that share a sample form a cluster:
//   stages 1-2  every block gathers its own token range into K-major operand tiles and contracts it on the
//               tensor core (tcgen05.mma, bf16 in / fp32 in tensor memory) into a PARTIAL k'_in x k'_out block;
//   exchange    block r of the cluster owns rows [r TM/NC, (r+1) TM/NC) of the sample's block: every block writes
//               those rows of its partial block from tensor memory straight into a receive area in the owner's
//               shared memory (distributed shared memory stores, posted: nobody waits for a remote load);
//   stage 3     after a cluster barrier the owner adds the NC partial slices it received, so that every entry of
//               Eq. 2's block is complete in exactly one thread block, hashes it from the seed (once per sample,
//               not once per token chunk) and adds it into its own k-bin accumulator;
//   reduce      slice r of the output row belongs to block r: every block writes the r-th slice of its
//               accumulator into the owner's second receive area, and after one more cluster barrier the owner
//               adds the NC slices and writes its part of the row with plain stores: no zero-fill, no global
//               atomics, and no thread block touches another's memory after the last barrier.
// The block must fit one TM x TN tile (k'_in, k'_out <= 128) and the accumulators must fit in shared memory;
// everything else takes the streaming kernel.
#include "factgrass_common.cuh"

#include <cooperative_groups.h>

#include <algorithm>

namespace cg = cooperative_groups;

namespace grass {

// Receive area for the partial blocks: NC slices (one per sender) of ROWS rows of TN floats; the 16-byte chunk
// cc of row r sits at chunk cc ^ (r & 7), so that the owner's 16-byte loads of consecutive chunks of a row touch
// every bank once per 128 bytes.
template <int TN>
__device__ __forceinline__ int recv_offset(int row, int c)
{
    return row * TN + ((((c >> 2) ^ (row & 7)) << 2) | (c & 3));
}

struct ProjectArgs {
    const float* recv;   // this thread block's receive area: NC slices of ROWS x TN floats
    float* bins;         // this thread block's k-bin accumulator
    int a_lo;            // first block row owned here
    int kin, kout;
    uint32_t k, s;
    uint64_t seed;
};

// Stage 3 in the owner: adds the NC partial slices, hashes every entry (flat position q = a*kout + c,
// input-major flattening) and adds it into the k-bin accumulator.
template <int TM, int TN, int NC>
__device__ __forceinline__ void sum_and_project(const ProjectArgs& x)
{
    constexpr int ROWS = TM / NC;                          // rows of C completed here
    constexpr int CPR = TN / 4;                            // 16-byte chunks per row
    constexpr int CHUNKS = ROWS * CPR;
    constexpr int E4 = (CHUNKS + kFgThreads - 1) / kFgThreads;   // chunks per thread
    static_assert(ROWS * NC == TM && ROWS >= 8, "even split");
    const int tid = threadIdx.x;
    const float scale = 1.0f / sqrtf((float)x.s);
#pragma unroll
    for (int j = 0; j < E4; ++j) {
        const int ch = j * kFgThreads + tid;
        if (ch >= CHUNKS) break;
        const int row = ch / CPR, cc = ch % CPR;
        const int off = row * TN + ((cc ^ (row & 7)) << 2);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int q = 0; q < NC; ++q) {
            const float4 v = *reinterpret_cast<const float4*>(x.recv + q * (ROWS * TN) + off);
            acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
        }
        const uint32_t a = (uint32_t)(x.a_lo + row), c0 = (uint32_t)(cc * 4);
        if ((int)a >= x.kin) continue;
        if (x.s == 1) {
            uint32_t bucket[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                // positions are below 2^32 here (at most 128 x 128), so the counter's high half is zero
                const uint64_t h = sjlt_hash_counter(x.seed, (uint64_t)(a * (uint32_t)x.kout + c0 + i + 1u));
                bucket[i] = ((int)(c0 + i) < x.kout && acc[i] != 0.0f) ? sjlt_bucket(h, x.k) : 0xFFFFFFFFu;
                acc[i] = sjlt_signed(h, acc[i]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (bucket[i] != 0xFFFFFFFFu) atomicAdd(x.bins + bucket[i], acc[i]);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if ((int)(c0 + i) >= x.kout || acc[i] == 0.0f) continue;
                const uint64_t q = (uint64_t)a * (uint64_t)x.kout + (uint64_t)(c0 + i);
                for (uint32_t r = 0; r < x.s; ++r) {
                    const uint64_t h = sjlt_hash_counter(x.seed, q * x.s + r + 1);
                    atomicAdd(x.bins + sjlt_bucket(h, x.k), sjlt_signed(h, acc[i]) * scale);
                }
            }
        }
    }
}

template <int TM, int TN>
__global__ void __launch_bounds__(kFgThreads, 1)
factgrass_cluster_kernel(const LayerDesc* __restrict__ descs, const __grid_constant__ LayerDesc single, int32_t T,
                         const int64_t* __restrict__ tok_begin, const int32_t* __restrict__ tok_count,
                         int32_t chunk_len, float* __restrict__ out, int64_t ld_out, uint32_t* dev_status,
                         int out_bf16)
{
    static_assert((TM == 64 && TN == 64) || (TM == 128 && TN == 128), "tile");
    constexpr int A_TILE = TM * (int)tc::ROW_BYTES, G_TILE = TN * (int)tc::ROW_BYTES;
    constexpr int STAGE = A_TILE + G_TILE;
    constexpr int NBUF = kFgBufs;
    constexpr int GA = kFgThreads / TM, GG = kFgThreads / TN;
    constexpr int PASS_A = 4 / GA, PASS_G = 4 / GG;
    constexpr uint32_t ACC_COLS = TN;
    constexpr int RECV_BYTES = TM * TN * 4;              // NC slices of (TM / NC) x TN floats

    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[NBUF + 1];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    // operand tiles | receive area for partial blocks | k bins | receive area for bin slices (NC x ceil(k / NC)).
    // The receive areas are written by the other thread blocks of the cluster at any time before the barriers,
    // so they overlap nothing.
    float* recv = reinterpret_cast<float*>(smem + NBUF * STAGE);
    float* bins = reinterpret_cast<float*>(smem + NBUF * STAGE + RECV_BYTES);

    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t nc = cluster.num_blocks(), rank = cluster.block_rank();
    // "I have started": the other half of this barrier is waited for just before the first write into another thread
    // block's shared memory, which is only defined once that thread block is running (by then everyone has arrived)
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    const LayerDesc& L = descs ? descs[blockIdx.z] : single;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.y;
    const int kin = L.kin, kout = L.kout;
    const int64_t d_in = L.d_in, d_out = L.d_out;
    const uint32_t k = L.k, s = L.s;
    const uint64_t seed = L.seed;
    const uint32_t per = (k + nc - 1) / nc;               // bins per slice of the output row
    float* recv_bins = bins + (k + 3) / 4 * 4;

    int Tb = T;
    if (tok_count) {
        Tb = __ldg(tok_count + b);
        if (Tb < 0 || Tb > T) {
            if (dev_status && tid == 0 && rank == 0) atomicOr(dev_status, GRASS_DEV_BAD_LENGTH);
            Tb = Tb < 0 ? 0 : T;
        }
    }
    const int64_t row0 = tok_begin ? __ldg(tok_begin + b) : (int64_t)b * T;
    const int t_begin = (int)rank * chunk_len;
    const int t_end = min(Tb, t_begin + chunk_len);
    // a thread block without tokens (short sample, empty factor mask) still takes part in every cluster step
    const bool work = t_begin < t_end && kin > 0 && kout > 0;

    // stage 1, first half: this thread's gather columns (fixed for the whole token range).  The mask loads are
    // issued before the set-up below so that their latency is hidden behind it.
    const int aL = tid % TM, gL = tid % TN;
    const int grpA = tid / TM, grpG = tid / TN;
    bool okA = work && aL < kin, okG = work && gL < kout;
    uint32_t colA = okA ? (L.mask_in ? __ldg(L.mask_in + aL) : (uint32_t)aL) : 0u;
    uint32_t colG = okG ? (L.mask_out ? __ldg(L.mask_out + gL) : (uint32_t)gL) : 0u;

    const uint32_t bar0 = tc::smem_u32(&bars[0]), bar_done = tc::smem_u32(&bars[NBUF]);
    if (tid == 0) {
        for (int i = 0; i < NBUF; ++i) tc::mbar_init(bar0 + 8 * i, 1);
        tc::mbar_init(bar_done, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(&tmem_slot)),
                     "r"(ACC_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    for (uint32_t i = tid; i < k; i += kFgThreads) bins[i] = 0.0f;
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_slot;

    bool ok = true, bad = false;
    if (work) {
        if (okA && colA >= (uint32_t)L.d_in) { bad = true; okA = false; colA = 0; }
        if (okG && colG >= (uint32_t)L.d_out) { bad = true; okG = false; colG = 0; }
        const uint16_t* pA = reinterpret_cast<const uint16_t*>(L.A) + row0 * d_in + colA;
        const uint16_t* pG = reinterpret_cast<const uint16_t*>(L.G) + row0 * d_out + colG;

        // Two register sets: the loads of the next 32-token step are already in flight while this step's
        // values are written to shared memory, so the memory pipe never runs empty between steps.
        uint32_t ra0[PASS_A][8], rg0[PASS_G][8], ra1[PASS_A][8], rg1[PASS_G][8];
        auto prefetch = [&](uint32_t (&ra)[PASS_A][8], uint32_t (&rg)[PASS_G][8], int t0) {
#pragma unroll
            for (int ps = 0; ps < PASS_A; ++ps)
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int t = t0 + (ps * GA + grpA) * 8 + i;
                    ra[ps][i] = (okA && t < t_end) ? (uint32_t)gather_u16(pA + (int64_t)t * d_in) : 0u;
                }
#pragma unroll
            for (int ps = 0; ps < PASS_G; ++ps)
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int t = t0 + (ps * GG + grpG) * 8 + i;
                    rg[ps][i] = (okG && t < t_end) ? (uint32_t)gather_u16(pG + (int64_t)t * d_out) : 0u;
                }
        };
        auto stash = [&](const uint32_t (&ra)[PASS_A][8], const uint32_t (&rg)[PASS_G][8], int buf) {
            unsigned char* sa = smem + buf * STAGE;
            unsigned char* sg = sa + A_TILE;
#pragma unroll
            for (int ps = 0; ps < PASS_A; ++ps)
                *reinterpret_cast<uint4*>(sa + tc::operand_chunk_offset(aL, ps * GA + grpA)) = pack8_bf16(ra[ps]);
#pragma unroll
            for (int ps = 0; ps < PASS_G; ++ps)
                *reinterpret_cast<uint4*>(sg + tc::operand_chunk_offset(gL, ps * GG + grpG)) = pack8_bf16(rg[ps]);
        };

        // stage 2: C += A'^T G' over this block's tokens, 32 per step
        const uint32_t smem_base = tc::smem_u32(smem);
        const uint32_t idesc = tc::make_idesc(TM, TN);
        auto step = [&](uint32_t (&ra)[PASS_A][8], uint32_t (&rg)[PASS_G][8], int t0, int it) {
            const int buf = it % NBUF;
            // the MMAs that read this buffer two steps ago must have finished before it is overwritten
            if (it >= NBUF) ok = tc::mbar_wait(bar0 + 8 * buf, (uint32_t)(it / NBUF - 1) & 1u) && ok;
            stash(ra, rg, buf);
            if (t0 + 2 * kTokTile < t_end) prefetch(ra, rg, t0 + 2 * kTokTile);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();
            if (tid == 0) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a0 = smem_base + buf * STAGE, g0 = a0 + A_TILE;
#pragma unroll
                for (int ks = 0; ks < kTokTile / 16; ++ks)
                    tc::umma_bf16(tmem_d, tc::make_smem_desc(a0 + ks * 32), tc::make_smem_desc(g0 + ks * 32), idesc,
                                  (it > 0 || ks > 0) ? 1u : 0u);
                tc::umma_commit(bar0 + 8 * buf);                       // buffer free once these MMAs have read it
                if (t0 + kTokTile >= t_end) tc::umma_commit(bar_done); // accumulator complete
            }
        };
        prefetch(ra0, rg0, t_begin);
        if (t_begin + kTokTile < t_end) prefetch(ra1, rg1, t_begin + kTokTile);
        for (int t0 = t_begin, it = 0; t0 < t_end; t0 += 2 * kTokTile, it += 2) {
            step(ra0, rg0, t0, it);
            if (t0 + kTokTile < t_end) step(ra1, rg1, t0 + kTokTile, it + 1);
        }
        ok = tc::mbar_wait(bar_done, 0) && ok;      // all MMAs done: accumulator complete, operand tiles free
        if (!ok) abort_flag = 1;
    }
    if (bad && dev_status) atomicOr(dev_status, GRASS_DEV_BAD_INDEX);
    __syncthreads();
    ok = abort_flag == 0;
    if (!ok && tid == 0 && dev_status) atomicOr(dev_status, GRASS_DEV_TIMEOUT);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    // exchange: the rows of the partial block go from tensor memory to their owners (zeros where there was no work).
    // Accumulator row a sits in tensor-memory lane a (TM = 128) or lane (a % 16) + 32 * (a / 16) (TM = 64);
    // warp w may read lanes 32 * (w % 4) .. + 31; the two warps that share a lane quarter split the columns.
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");     // every thread block of the cluster runs
    const bool nc_ok = nc == 1 || nc == 2 || nc == 4 || nc == 8;    // the launcher forms no other clusters
    const int rows = TM / (int)(nc_ok ? nc : 1);
    if (nc_ok) {
        const int quarter = warp & 3;
        const uint32_t tq = tmem_d + ((uint32_t)(quarter * 32) << 16);
        const bool have = work && ok;
        if constexpr (TM == 64) {
            const int c0 = (warp >> 2) * 32;
            uint32_t v[16];
            if (have) {
                tc::tmem_ld_16x256b_x4(tq + (uint32_t)c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = 0u;
            }
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
                const int a = quarter * 16 + (lane >> 2) + 8 * ((e & 3) >> 1);
                const int c = c0 + 8 * (e >> 2) + 2 * (lane & 3);
                float* dst = cluster.map_shared_rank(recv, a / rows) + (int)rank * (rows * TN);
                *reinterpret_cast<uint2*>(dst + recv_offset<TN>(a % rows, c)) = make_uint2(v[e], v[e + 1]);
            }
        } else {
            const int a = quarter * 32 + lane;
            float* dst = cluster.map_shared_rank(recv, a / rows) + (int)rank * (rows * TN);
#pragma unroll 1
            for (int c0 = (warp >> 2) * 32; c0 < TN; c0 += 64) {
                uint32_t v[32];
                if (have) {
                    tc::tmem_ld32(tq + (uint32_t)c0, v);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = 0u;
                }
#pragma unroll
                for (int e = 0; e < 32; e += 4)
                    *reinterpret_cast<uint4*>(dst + recv_offset<TN>(a % rows, c0 + e)) =
                        make_uint4(v[e], v[e + 1], v[e + 2], v[e + 3]);
            }
        }
    } else if (tid == 0 && dev_status) {
        atomicOr(dev_status, GRASS_DEV_TIMEOUT);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(ACC_COLS) : "memory");
    }
    cluster.sync();      // every thread block holds the NC partial slices of its rows

    // stage 3 in the owner of the rows
    {
        const ProjectArgs pa{recv, bins, (int)rank * rows, kin, kout, k, s, seed};
        switch (nc) {
            case 1: sum_and_project<TM, TN, 1>(pa); break;
            case 2: sum_and_project<TM, TN, 2>(pa); break;
            case 4: sum_and_project<TM, TN, 4>(pa); break;
            case 8: sum_and_project<TM, TN, 8>(pa); break;
            default: break;
        }
    }
    __syncthreads();     // this thread block's accumulator is final

    // reduce: slice o of the accumulator goes to thread block o's second receive area ...
    if (nc_ok) {
        for (uint32_t i = tid; i < k; i += kFgThreads) {
            const uint32_t o = i / per;
            cluster.map_shared_rank(recv_bins, o)[rank * per + (i - o * per)] = bins[i];
        }
    }
    cluster.sync();      // ... and after this barrier nobody touches another thread block's memory
    if (nc_ok) {
        const int64_t orow = (int64_t)b * ld_out + L.out_offset;
        const uint32_t lo = rank * per, hi = min(lo + per, k);
        for (uint32_t i = lo + tid; i < hi; i += kFgThreads) {
            float acc = 0.0f;
            for (uint32_t q = 0; q < nc; ++q) acc += recv_bins[q * per + (i - lo)];
            store_out(out, orow + i, acc, out_bf16);
        }
    }
}

static size_t cluster_smem_bytes(int tile, uint32_t max_k)
{
    const size_t stage = 2 * (size_t)tile * tc::ROW_BYTES;
    const size_t recv = (size_t)tile * tile * 4;
    const size_t bins = ((size_t)max_k + 3) / 4 * 4 * sizeof(float);
    const size_t recv_bins = ((size_t)max_k + 8) * sizeof(float);       // NC * ceil(k / NC) <= k + NC - 1
    return kFgBufs * stage + recv + bins + recv_bins;
}

bool cluster_path_fits(const LayerDesc* d, int32_t L, ClusterPlan* plan)
{
    int max_kk = 0;
    uint32_t max_k = 0;
    for (int l = 0; l < L; ++l) {
        max_kk = std::max(max_kk, std::max(d[l].kin, d[l].kout));
        max_k = std::max(max_k, d[l].k);
    }
    if (max_kk > 128) return false;
    const int tile = max_kk > 64 ? 128 : 64;
    plan->tile_m = plan->tile_n = tile;
    plan->smem = cluster_smem_bytes(tile, max_k);
    if (plan->smem + 2048 > 200 * 1024) return false;
    // resident thread blocks per SM: registers, `tile` tensor-memory columns, shared memory; at most 164 KB of
    // the SM go to shared memory, so that the gathered loads in flight keep their L1
    cudaFuncAttributes fa;
    const cudaError_t e = tile == 64 ? cudaFuncGetAttributes(&fa, factgrass_cluster_kernel<64, 64>)
                                     : cudaFuncGetAttributes(&fa, factgrass_cluster_kernel<128, 128>);
    if (e != cudaSuccess || fa.numRegs <= 0) return false;
    int per_sm = std::min(65536 / (fa.numRegs * kFgThreads), 512 / tile);
    per_sm = std::min<int>(per_sm, (int)((164 * 1024) / (plan->smem + 1024 + 64)));
    plan->per_sm = per_sm;
    return per_sm >= 1;
}

grass_status launch_factgrass_cluster(const LayerDesc* dev_descs, const LayerDesc& single, const ClusterPlan& plan,
                                      int32_t L, int32_t B, int32_t T, const int64_t* tok_begin,
                                      const int32_t* tok_count, int32_t nc, int32_t chunk_len, float* out,
                                      int64_t ld_out, uint32_t* dev_status, cudaStream_t st, int out_bf16)
{
    auto launch = [&](auto kern) -> grass_status {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem) != cudaSuccess)
            return GRASS_ERR_CUDA;
        int carve = 100;
        {
            const size_t need = (size_t)plan.per_sm * (plan.smem + 1024 + 64);
            const int configs_kb[] = {8, 16, 32, 64, 100, 132, 164, 196, 228};
            for (int kb : configs_kb)
                if ((size_t)kb * 1024 >= need) { carve = (kb * 100 + 227) / 228; break; }
        }
        carve = (int)tuning(GRASS_TUNE_FACTGRASS_CARVEOUT, carve);
        if (cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, carve) != cudaSuccess)
            return GRASS_ERR_CUDA;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)nc, (unsigned)B, (unsigned)L);
        cfg.blockDim = dim3(kFgThreads, 1, 1);
        cfg.dynamicSmemBytes = plan.smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)nc;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, kern, dev_descs, single, T, tok_begin, tok_count, chunk_len, out,
                                           ld_out, dev_status, out_bf16);
        return e == cudaSuccess ? launch_status() : GRASS_ERR_CUDA;
    };
    if (plan.tile_m == 64) return launch(factgrass_cluster_kernel<64, 64>);
    return launch(factgrass_cluster_kernel<128, 128>);
}

}  // namespace grass
