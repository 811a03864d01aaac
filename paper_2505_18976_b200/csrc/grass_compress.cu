// grass_compress: Mask_k' gather fused with the SJLT_k scatter-add (GraSS, Section 3.3.1).
//
// One CTA owns S samples and a contiguous range of masked positions j.  Each thread reads the
// mask index of its j once, derives (bucket, sign) once from the seed, and applies them to the S
// samples: S independent gathered loads per j are in flight together, consecutive lanes hold
// consecutive (ascending) indices so the loads of a warp fall into the fewest 32-byte sectors.
// Non-zero values are added into a per-sample k-bin accumulator in shared memory; exact zeros are
// skipped (the input sparsity the paper's Section 3.1 builds on).  When the positions of a sample are
// split over up to 8 CTAs, those CTAs form a thread-block cluster and add their bins through distributed
// shared memory, each CTA storing one slice of the row: no zero-fill pass and no global atomics.  Wider
// splits (few samples, very long masks) fall back to a zero-fill plus global reductions.
// With the identity mask on vector-aligned rows (plain SJLT) the rows are streamed with 16-byte loads instead
// of gathers.  grass_mask (Mask alone, Section 3.2) is the gather without the projection.
#include "grass_common.cuh"
#include "tcgen05_util.cuh"

#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace grass {

constexpr int kThreads = 256;
// Dense rows with many zeros: the non-zero entries of a warp's round of loads are first compacted into a small
// per-warp queue in shared memory, so that every lane hashes a non-zero (the cost of the projection follows the
// non-zeros, Section 3.1) instead of the whole warp waiting on the lanes that hold one.
constexpr int kQueueCap = 128;                                  // entries per warp; fuller rounds are hashed in place
// an entry = the value and a 16-bit key: (position within the round) * 8 + sample of the CTA
constexpr int kQueueBytes = (kThreads / 32) * kQueueCap * (int)(sizeof(float) + sizeof(uint16_t));

// four consecutive elements of a row with one vector load (16 bytes of fp32, 8 bytes of bf16)
__device__ __forceinline__ void load4(const float* p, float (&v)[4])
{
    const float4 t = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&v)[4])
{
    const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
    v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xFFFF0000u);
    v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xFFFF0000u);
}

// DENSE: identity mask on vector-aligned rows (plain SJLT, the k' = p case of Section 3.3.1).  Rows are then
// streamed with vector loads, four consecutive positions per thread, and S > 1 samples share each hash.
// NT: threads per CTA (the gather path runs with 256 or 512; the streamed path always with kThreads).
template <typename T, int S, int U, bool S1, bool DENSE, int NT>
__global__ void __launch_bounds__(NT, DENSE ? 4 : (U >= 16 ? 1024 : 2048) / NT)
grass_compress_kernel(const T* __restrict__ g, int64_t n, int64_t p, int64_t ld,
                      const uint32_t* __restrict__ idx, int64_t kprime, uint32_t k, uint32_t s,
                      uint64_t seed, float scale, float* __restrict__ out, int64_t ld_out,
                      int64_t j_per_cta, int accumulate, int use_smem, uint32_t* dev_status, int out_bf16,
                      uint32_t idx_smem_bytes)
{
    extern __shared__ float bins[];  // S * k when use_smem
    const int tid = threadIdx.x;
    constexpr int nthr = NT;
    static_assert(!DENSE || NT == kThreads, "the streamed path is written for kThreads threads");
    const int64_t i0 = (int64_t)blockIdx.x * S;
    const int ns = (int)((n - i0) < (int64_t)S ? (n - i0) : (int64_t)S);
    const int64_t j0 = (int64_t)blockIdx.y * j_per_cta;
    const int64_t j1 = (j0 + j_per_cta) < kprime ? (j0 + j_per_cta) : kprime;

    // Whole-row thread blocks keep the index list in shared memory (idx_smem_bytes > 0: one bulk copy, started
    // before anything else): every thread block of the launch reads the whole list, and hundreds of them asking L2
    // for the same few lines at once take microseconds to be served.
    __shared__ __align__(8) unsigned long long idx_bar;
    uint32_t* sidx = reinterpret_cast<uint32_t*>(bins + (use_smem ? ((size_t)S * k + 3) / 4 * 4 : 0));
    const uint32_t idx_bulk = idx_smem_bytes ? (uint32_t)((kprime * 4) & ~(int64_t)15) : 0u;
    if (idx_smem_bytes && tid == 0) {
        const uint32_t bar = tc::smem_u32(&idx_bar);
        tc::mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (idx_bulk > 0) {
            tc::expect_tx(bar, idx_bulk);
            tc::bulk_copy(tc::smem_u32(sidx), idx, idx_bulk, bar);
        }
    }
    if (use_smem)
        for (uint32_t i = tid; i < (uint32_t)S * k; i += nthr) bins[i] = 0.0f;
    if (idx_smem_bytes)
        for (int64_t j = idx_bulk / 4 + tid; j < kprime; j += nthr) sidx[j] = __ldg(idx + j);   // at most 3 entries
    if (use_smem || idx_smem_bytes) __syncthreads();
    // the list has landed; should the bounded wait expire, the indices are read from global memory after all
    // (after one more bounded wait: no copy may be in flight into shared memory that is about to be reused or left)
    bool idx_in_smem = idx_smem_bytes != 0;
    if (idx_bulk > 0 && !tc::mbar_wait(tc::smem_u32(&idx_bar), 0)) {
        idx_in_smem = false;
        if (tid == 0 && dev_status) atomicOr(dev_status, GRASS_DEV_TIMEOUT);
        tc::mbar_wait(tc::smem_u32(&idx_bar), 0);
    }

    const T* rows[S];
#pragma unroll
    for (int si = 0; si < S; ++si) rows[si] = g + (i0 + (si < ns ? si : 0)) * ld;

    bool bad = false;
    if constexpr (DENSE) {
        constexpr int UD = S >= 8 ? 1 : 8 / S;     // vector loads per sample in flight per thread (8 in all)
        const int lane = tid & 31, warp = tid >> 5;
        // this warp's queue, behind the bins (8-byte aligned)
        unsigned char* qbase = reinterpret_cast<unsigned char*>(bins) +
                               (use_smem ? (((size_t)S * k * sizeof(float) + 7) & ~(size_t)7) : 0);
        float* qval = reinterpret_cast<float*>(qbase) + warp * kQueueCap;
        uint16_t* qkey = reinterpret_cast<uint16_t*>(qbase + (kThreads / 32) * kQueueCap * sizeof(float)) + warp * kQueueCap;
        static_assert(kThreads * 4 * UD * 8 <= 65536 && S <= 8, "queue key is 16 bits");
        // the trip count is the same for every thread (the warp votes below); positions beyond j1 load as zeros
        for (int64_t round0 = j0; round0 < j1; round0 += (int64_t)kThreads * 4 * UD) {
            const int64_t jb = round0 + (int64_t)tid * 4;
            float v[UD][S][4];
#pragma unroll
            for (int u = 0; u < UD; ++u) {
                const int64_t j = jb + (int64_t)u * kThreads * 4;
#pragma unroll
                for (int si = 0; si < S; ++si) {
                    if (si < ns && j + 3 < j1) {
                        load4(rows[si] + j, v[u][si]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            v[u][si][e] = (si < ns && j + e < j1) ? elem<T>::load(rows[si] + j + e) : 0.0f;
                    }
                }
            }
            // Non-zeros of this round: per lane, then over the warp.  The first vector of every lane is counted
            // first: where that sample already says the round is too full for the queue, the exact count is skipped.
            bool queue = false;
            uint32_t cnt = 0, total = 0;
#pragma unroll
            for (int si = 0; si < S; ++si)
#pragma unroll
                for (int e = 0; e < 4; ++e) cnt += (v[0][si][e] != 0.0f) ? 1u : 0u;
            if (__reduce_add_sync(0xFFFFFFFFu, cnt) * UD <= 2u * kQueueCap) {
#pragma unroll
                for (int u = 1; u < UD; ++u)
#pragma unroll
                    for (int si = 0; si < S; ++si)
#pragma unroll
                        for (int e = 0; e < 4; ++e) cnt += (v[u][si][e] != 0.0f) ? 1u : 0u;
                total = __reduce_add_sync(0xFFFFFFFFu, cnt);
                if (total == 0) continue;
                queue = total <= (uint32_t)kQueueCap;
            }
            if (queue) {
                uint32_t incl = cnt;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                    if (lane >= d) incl += t;
                }
                uint32_t at = incl - cnt;
#pragma unroll
                for (int u = 0; u < UD; ++u)
#pragma unroll
                    for (int si = 0; si < S; ++si)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float x = v[u][si][e];
                            if (x != 0.0f) {
                                qval[at] = x;
                                qkey[at] = (uint16_t)(((tid * 4 + u * kThreads * 4 + e) << 3) | si);
                                ++at;
                            }
                        }
                __syncwarp();
                for (uint32_t q = lane; q < total; q += 32) {
                    const uint32_t key = qkey[q];
                    const uint32_t si = key & 7u;
                    const float x = qval[q];
                    const uint64_t pos = (uint64_t)(round0 + (int64_t)(key >> 3));
                    const uint32_t draws = S1 ? 1u : s;
                    for (uint32_t r = 0; r < draws; ++r) {
                        const uint64_t h = sjlt_hash_counter(seed, S1 ? (pos + 1) : (pos * s + r + 1));
                        const uint32_t b = sjlt_bucket(h, k);
                        const float sx = S1 ? sjlt_signed(h, x) : sjlt_signed(h, x) * scale;
                        if (use_smem) atomicAdd(&bins[si * k + b], sx);
                        else atomicAdd(out + (i0 + si) * ld_out + b, sx);
                    }
                }
                __syncwarp();       // the queue is rewritten in the next round
                continue;
            }
#pragma unroll
            for (int u = 0; u < UD; ++u) {
                const int64_t j = jb + (int64_t)u * kThreads * 4;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    bool any = false;
#pragma unroll
                    for (int si = 0; si < S; ++si) any = any || (v[u][si][e] != 0.0f);
                    if (!any) continue;     // the cost of the projection follows the non-zeros (Section 3.1)
                    const uint64_t pos = (uint64_t)(j + e);
                    const uint32_t draws = S1 ? 1u : s;
                    for (uint32_t r = 0; r < draws; ++r) {
                        const uint64_t h = sjlt_hash_counter(seed, S1 ? (pos + 1) : (pos * s + r + 1));
                        const uint32_t b = sjlt_bucket(h, k);
#pragma unroll
                        for (int si = 0; si < S; ++si) {
                            const float x = v[u][si][e];
                            if (x != 0.0f) {
                                const float sx = S1 ? sjlt_signed(h, x) : sjlt_signed(h, x) * scale;
                                if (use_smem) atomicAdd(&bins[(uint32_t)si * k + b], sx);
                                else atomicAdd(out + (i0 + si) * ld_out + b, sx);
                            }
                        }
                    }
                }
            }
        }
    } else
    // the trip count is the same for every lane of a warp (the warp votes below)
    for (int64_t jw = j0 + (tid & ~31); jw < j1; jw += (int64_t)nthr * U) {
        const int64_t jb = jw + (tid & 31);
        uint32_t col[U];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t j = jb + (int64_t)u * nthr;
            ok[u] = j < j1;
            uint32_t c = 0;
            if (ok[u]) c = idx_in_smem ? sidx[j] : (idx ? __ldg(idx + j) : (uint32_t)j);
            if ((int64_t)c >= p) { bad = bad || ok[u]; ok[u] = false; c = 0; }
            col[u] = c;
        }
        float v[U][S];
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int si = 0; si < S; ++si)
                v[u][si] = (ok[u] && si < ns) ? elem<T>::load(rows[si] + col[u]) : 0.0f;

        if constexpr (S == 1) {
            // The cost of the projection follows the non-zeros (Section 3.1).  A lane hashes its own non-zero
            // entries one after the other, so the warp makes as many passes as its fullest lane has non-zeros
            // (three or four of eight at 90 % zeros) instead of one per loaded entry.
            uint32_t pending = 0;
#pragma unroll
            for (int u = 0; u < U; ++u) pending |= (ok[u] && v[u][0] != 0.0f) ? (1u << u) : 0u;
            while (__any_sync(0xFFFFFFFFu, pending != 0)) {
                if (pending != 0) {
                    const int u = __ffs((int)pending) - 1;
                    pending &= pending - 1;
                    float x = v[0][0];
#pragma unroll
                    for (int t = 1; t < U; ++t) x = (u == t) ? v[t][0] : x;
                    const uint64_t j = (uint64_t)(jb + (int64_t)u * nthr);
                    const uint32_t draws = S1 ? 1u : s;
                    for (uint32_t r = 0; r < draws; ++r) {
                        const uint64_t h = sjlt_hash_counter(seed, S1 ? (j + 1) : (j * s + r + 1));
                        const uint32_t b = sjlt_bucket(h, k);
                        const float sx = S1 ? sjlt_signed(h, x) : sjlt_signed(h, x) * scale;
                        if (use_smem) atomicAdd(&bins[b], sx);
                        else atomicAdd(out + i0 * ld_out + b, sx);
                    }
                }
            }
        } else {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (!ok[u]) continue;
                // the hash is shared by the samples of the thread block: it is computed where any of them has a
                // non-zero entry
                bool any = false;
#pragma unroll
                for (int si = 0; si < S; ++si) any = any || (v[u][si] != 0.0f);
                if (!any) continue;
                const uint64_t j = (uint64_t)(jb + (int64_t)u * nthr);
                const uint32_t draws = S1 ? 1u : s;
                for (uint32_t r = 0; r < draws; ++r) {
                    const uint64_t h = sjlt_hash_counter(seed, S1 ? (j + 1) : (j * s + r + 1));
                    const uint32_t b = sjlt_bucket(h, k);
#pragma unroll
                    for (int si = 0; si < S; ++si) {
                        const float x = v[u][si];
                        if (x != 0.0f) {
                            const float sx = S1 ? sjlt_signed(h, x) : sjlt_signed(h, x) * scale;
                            if (use_smem) atomicAdd(&bins[(uint32_t)si * k + b], sx);
                            else atomicAdd(out + (i0 + si) * ld_out + b, sx);
                        }
                    }
                }
            }
        }
    }
    if (bad && dev_status) atomicOr(dev_status, GRASS_DEV_BAD_INDEX);

    if (use_smem && accumulate == 2) {
        // the gridDim.y CTAs that share these samples are one cluster: rank r sums slice r of every
        // CTA's bins over distributed shared memory and stores it
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();
        const uint32_t nr = cluster.num_blocks(), r = cluster.block_rank();
        const uint32_t per = (k + nr - 1) / nr;
        const uint32_t lo = r * per, hi = (lo + per) < k ? (lo + per) : k;
        for (int si = 0; si < ns; ++si) {
            for (uint32_t i = lo + tid; i < hi; i += nthr) {
                float acc = 0.0f;
                for (uint32_t q = 0; q < nr; ++q) acc += cluster.map_shared_rank(bins, q)[(uint32_t)si * k + i];
                store_out(out, (i0 + si) * ld_out + i, acc, out_bf16);
            }
        }
        cluster.sync();  // nobody leaves while its bins may still be read
    } else if (use_smem) {
        __syncthreads();
        for (int si = 0; si < ns; ++si) {
            float* dst = out + (i0 + si) * ld_out;
            const float* src = bins + (uint32_t)si * k;
            if (accumulate) {
                for (uint32_t i = tid; i < k; i += nthr) {
                    const float x = src[i];
                    if (x != 0.0f) atomicAdd(dst + i, x);
                }
            } else {
                for (uint32_t i = tid; i < k; i += nthr) store_out(out, (i0 + si) * ld_out + i, src[i], out_bf16);
            }
        }
    }
}

// Stand-alone Mask_k' (Section 3.2): out[i, j] = g[i, idx[j]], written as fp32.
template <typename T>
__global__ void __launch_bounds__(kThreads)
grass_mask_kernel(const T* __restrict__ g, int64_t p, int64_t ld, const uint32_t* __restrict__ idx, int64_t kprime,
                  float* __restrict__ out, int64_t ld_out, uint32_t* dev_status)
{
    const int64_t i = blockIdx.y;
    const T* row = g + i * ld;
    float* orow = out + i * ld_out;
    bool bad = false;
    for (int64_t j = (int64_t)blockIdx.x * kThreads * 4 + threadIdx.x; j < kprime && j < ((int64_t)blockIdx.x + 1) * kThreads * 4;
         j += kThreads) {
        const uint32_t c = __ldg(idx + j);
        if ((int64_t)c >= p) { bad = true; orow[j] = 0.0f; continue; }
        orow[j] = elem<T>::load(row + c);
    }
    if (bad && dev_status) atomicOr(dev_status, GRASS_DEV_BAD_INDEX);
}

struct CompressPlan {
    int dense;      // identity mask on vector-aligned rows: streamed with vector loads
    int S;          // samples per CTA
    int jsplit;     // CTAs that share one sample group (split of the masked positions)
    int use_smem;   // k-bin accumulators fit in shared memory
    int cluster;    // the jsplit CTAs are one thread-block cluster (DSMEM reduction)
    int out_bf16;   // rows are stored as bf16 (final store only)
    uint32_t idx_smem;  // bytes of shared memory for a copy of the index list (0: indices are read from global memory)
    int threads;    // threads per CTA of the gather path (256 or 512)
    int U;          // gathered loads in flight per thread and sample
};

static CompressPlan plan_compress(int64_t n, int64_t kprime, uint32_t k, int sm_count, bool dense)
{
    CompressPlan pl;
    pl.dense = dense;
    const size_t bin_bytes = (size_t)k * sizeof(float);
    const size_t smem_cap = 200 * 1024;
    pl.use_smem = bin_bytes <= smem_cap;
    // One sample per CTA: the hash is a few dozen integer instructions per position, far below what the
    // gathered loads leave idle, so sharing it between samples buys nothing and costs occupancy.
    // Dense rows are the exception: every position is read, the hash is the larger cost, and two samples share it
    // where their bins still leave room for several CTAs per SM (four samples measured slower at k = 4,096).
    int S = (int)tuning(GRASS_TUNE_COMPRESS_SAMPLES, dense && bin_bytes * 2 <= 64 * 1024 ? 2 : 1);
    if (S != 1 && S != 2 && S != 4 && S != 8) S = 1;
    while (S > 1 && pl.use_smem && bin_bytes * S > smem_cap) S >>= 1;
    if (!pl.use_smem) S = 1;
    pl.S = S;
    int U = S == 1 ? 8 : (S == 8 ? 2 : 4);
    if (S == 1 && !dense && tuning(GRASS_TUNE_COMPRESS_LOADS, 8) == 16) U = 16;
    pl.U = U;
    const int64_t groups = (n + S - 1) / S;
    pl.threads = kThreads;
    if (!dense) {
        // With a row for every SM, a thread block of up to 1,024 threads takes a whole row in one round of loads:
        // no position split, so no cluster, no exchange of bins and no thread blocks left waiting for a slot
        // (config 1: 25.2 -> 22.9 us).  Longer masks and fewer rows keep 256 threads and split the positions.
        int t = kThreads;
        if (S == 1 && groups >= sm_count && kprime <= (int64_t)4 * kThreads * U)
            while ((int64_t)t * U < kprime) t *= 2;
        t = (int)tuning(GRASS_TUNE_COMPRESS_THREADS, t);
        if (t == 2 * kThreads || t == 4 * kThreads) pl.threads = t;
    }
    // split positions until there are ~4 CTAs per SM, but keep one full round of loads per CTA
    const int64_t round = (int64_t)pl.threads * U;
    const int64_t max_js = kprime / round > 0 ? kprime / round : 1;
    int64_t js = 1;
    while (js < 8 && groups * js < (int64_t)sm_count * 4 && js * 2 <= max_js) js *= 2;
    pl.cluster = 1;
    if (groups * js < sm_count && js * 2 <= max_js) {
        // very few samples: split wider than a cluster allows and reduce with global atomics
        js = ((int64_t)sm_count * 2 + groups - 1) / groups;
        if (js > max_js) js = max_js;
        pl.cluster = 0;
    }
    const int forced = (int)tuning(GRASS_TUNE_COMPRESS_JSPLIT, 0);
    if (forced > 0) {
        js = forced;
        pl.cluster = forced <= 8 && tuning(GRASS_TUNE_COMPRESS_CLUSTER, 1) != 0;
    }
    if (js < 1) js = 1;
    if (js > 65535) js = 65535;
    if (js == 1 || !pl.use_smem) pl.cluster = 0;
    pl.jsplit = (int)js;
    return pl;
}

template <typename T, int S, int U>
static grass_status launch_compress(const T* g, int64_t n, int64_t p, int64_t ld, const uint32_t* idx,
                                    int64_t kprime, const grass_sjlt_spec& sp, float* out, int64_t ld_out,
                                    const CompressPlan& pl, uint32_t* dev_status, cudaStream_t st)
{
    const int64_t groups = (n + S - 1) / S;
    int64_t j_per_cta = (kprime + pl.jsplit - 1) / pl.jsplit;
    if (pl.dense) j_per_cta = (j_per_cta + 3) / 4 * 4;      // vector loads start on multiples of four positions
    // 0: one CTA owns the row, plain stores; 1: global reductions into a zeroed row; 2: cluster reduction
    const int accumulate = pl.cluster ? 2 : ((pl.jsplit > 1 || !pl.use_smem) ? 1 : 0);
    size_t smem = pl.use_smem ? (size_t)S * sp.k * sizeof(float) : 0;
    if (pl.dense) smem = ((smem + 7) & ~(size_t)7) + kQueueBytes;      // the warps' non-zero queues
    if (pl.idx_smem) smem = (smem + 15) / 16 * 16 + pl.idx_smem;       // a copy of the index list
    const float scale = 1.0f / sqrtf((float)sp.s);
    auto launch = [&](auto kern) -> grass_status {
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return GRASS_ERR_CUDA;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)groups, (unsigned)pl.jsplit, 1);
        cfg.blockDim = dim3((unsigned)(pl.dense ? kThreads : pl.threads), 1, 1);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        if (pl.cluster) {
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 1;
            attr[0].val.clusterDim.y = (unsigned)pl.jsplit;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
        }
        const int use_smem = pl.use_smem;
        cudaError_t e = cudaLaunchKernelEx(&cfg, kern, g, n, p, ld, idx, kprime, sp.k, sp.s, sp.seed, scale, out,
                                           ld_out, j_per_cta, accumulate, use_smem, dev_status, pl.out_bf16, pl.idx_smem);
        return e == cudaSuccess ? launch_status() : GRASS_ERR_CUDA;
    };
    if (pl.dense) {
        if (sp.s == 1) return launch(grass_compress_kernel<T, S, U, true, true, kThreads>);
        return launch(grass_compress_kernel<T, S, U, false, true, kThreads>);
    }
    if (pl.threads == 2 * kThreads) {
        if (sp.s == 1) return launch(grass_compress_kernel<T, S, U, true, false, 2 * kThreads>);
        return launch(grass_compress_kernel<T, S, U, false, false, 2 * kThreads>);
    }
    if (pl.threads == 4 * kThreads) {
        if (sp.s == 1) return launch(grass_compress_kernel<T, S, U, true, false, 4 * kThreads>);
        return launch(grass_compress_kernel<T, S, U, false, false, 4 * kThreads>);
    }
    if (sp.s == 1) return launch(grass_compress_kernel<T, S, U, true, false, kThreads>);
    return launch(grass_compress_kernel<T, S, U, false, false, kThreads>);
}

template <typename T>
static grass_status dispatch_compress(const T* g, int64_t n, int64_t p, int64_t ld, const uint32_t* idx,
                                      int64_t kprime, const grass_sjlt_spec& sp, float* out, int64_t ld_out,
                                      uint32_t* dev_status, cudaStream_t st, int out_bf16)
{
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return GRASS_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GRASS_ERR_CUDA;
    const bool dense = idx == nullptr && tuning(GRASS_TUNE_COMPRESS_DENSE, 1) != 0 &&
                       (uintptr_t)g % (4 * sizeof(T)) == 0 && ld % 4 == 0;
    CompressPlan pl = plan_compress(n, kprime, sp.k, sms, dense);
    pl.out_bf16 = out_bf16;
    // whole-row thread blocks, one for every SM or more: the index list (up to 48 KB) goes into shared memory
    pl.idx_smem = 0;
    if (!dense && idx && pl.jsplit == 1 && pl.S == 1 && pl.use_smem && n >= sms && kprime * 4 <= 48 * 1024 &&
        (uintptr_t)idx % 16 == 0 && tuning(GRASS_TUNE_COMPRESS_IDX_SMEM, 1) != 0)
        pl.idx_smem = (uint32_t)((kprime * 4 + 15) / 16 * 16);
    if (out_bf16 && !pl.cluster && (pl.jsplit > 1 || !pl.use_smem)) {
        // a bf16 row is rounded once, at the final store, so it needs a launch shape in which one thread block
        // or one cluster owns the row: no partial sums in global memory
        if (!pl.use_smem) return GRASS_ERR_UNSUPPORTED;
        pl.jsplit = pl.jsplit > 8 ? 8 : pl.jsplit;
        pl.cluster = pl.jsplit > 1;
    }
    if (!pl.cluster && (pl.jsplit > 1 || !pl.use_smem)) {
        cudaError_t e = cudaMemset2DAsync(out, (size_t)ld_out * sizeof(float), 0, (size_t)sp.k * sizeof(float),
                                          (size_t)n, st);
        if (e != cudaSuccess) return GRASS_ERR_CUDA;
    }
    switch (pl.S) {
        case 8: return launch_compress<T, 8, 2>(g, n, p, ld, idx, kprime, sp, out, ld_out, pl, dev_status, st);
        case 4: return launch_compress<T, 4, 4>(g, n, p, ld, idx, kprime, sp, out, ld_out, pl, dev_status, st);
        case 2: return launch_compress<T, 2, 4>(g, n, p, ld, idx, kprime, sp, out, ld_out, pl, dev_status, st);
        default:
            if (pl.U == 16)
                return launch_compress<T, 1, 16>(g, n, p, ld, idx, kprime, sp, out, ld_out, pl, dev_status, st);
            return launch_compress<T, 1, 8>(g, n, p, ld, idx, kprime, sp, out, ld_out, pl, dev_status, st);
    }
}

}  // namespace grass

extern "C" grass_status grass_mask(const void* g, grass_dtype dt, int64_t n, int64_t p, int64_t ld, const uint32_t* idx,
                                   int64_t kprime, float* out, int64_t ld_out, uint32_t* dev_status, void* stream)
{
    if (n < 0 || p < 0 || kprime < 0 || kprime > p || ld < p || ld_out < kprime) return GRASS_ERR_INVALID_ARG;
    if (p >= 0xFFFFFFFFLL || n > 65535) return n > 65535 ? GRASS_ERR_UNSUPPORTED : GRASS_ERR_INVALID_ARG;
    if (dt != GRASS_F32 && dt != GRASS_BF16) return GRASS_ERR_UNSUPPORTED;
    if (n == 0 || kprime == 0) return GRASS_OK;
    if (!g || !idx || !out) return GRASS_ERR_INVALID_ARG;
    dim3 grid((unsigned)((kprime + grass::kThreads * 4 - 1) / (grass::kThreads * 4)), (unsigned)n);
    cudaStream_t st = (cudaStream_t)stream;
    if (dt == GRASS_F32)
        grass::grass_mask_kernel<float><<<grid, grass::kThreads, 0, st>>>((const float*)g, p, ld, idx, kprime, out, ld_out,
                                                                          dev_status);
    else
        grass::grass_mask_kernel<__nv_bfloat16><<<grid, grass::kThreads, 0, st>>>((const __nv_bfloat16*)g, p, ld, idx,
                                                                                  kprime, out, ld_out, dev_status);
    return grass::launch_status();
}

extern "C" grass_status grass_compress_out(const void* g, grass_dtype dt, int64_t n, int64_t p, int64_t ld,
                                           const uint32_t* idx, int64_t kprime, const grass_sjlt_spec* spec,
                                           void* out_v, grass_dtype out_dt, int64_t ld_out, uint32_t* dev_status,
                                           void* stream)
{
    if (!spec || spec->k == 0 || spec->s == 0) return GRASS_ERR_INVALID_ARG;
    if (n < 0 || p < 0 || kprime < 0 || kprime > p || ld < p || ld_out < (int64_t)spec->k) return GRASS_ERR_INVALID_ARG;
    if (p >= 0xFFFFFFFFLL) return GRASS_ERR_INVALID_ARG;
    if (!idx && kprime != p && kprime != 0) return GRASS_ERR_INVALID_ARG;
    if (dt != GRASS_F32 && dt != GRASS_BF16) return GRASS_ERR_UNSUPPORTED;
    if (out_dt != GRASS_F32 && out_dt != GRASS_BF16) return GRASS_ERR_UNSUPPORTED;
    if (n == 0) return GRASS_OK;
    if (!out_v || (!g && kprime > 0)) return GRASS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int out_bf16 = out_dt == GRASS_BF16;
    const size_t osz = out_bf16 ? 2 : 4;
    float* out = (float*)out_v;     // the kernels index it as fp32 or bf16 at the final store (store_out)
    if (kprime == 0) {
        return grass::cuda_ok(cudaMemset2DAsync(out, (size_t)ld_out * osz, 0, (size_t)spec->k * osz, (size_t)n, st));
    }
    // Row staging for dense masks (grass_compress_rows.cu): whole rows through shared memory, window by window,
    // the masked elements picked from there.  It is built and parity-tested but not chosen automatically: on B200
    // it is slower than the gathers below even where the mask touches nine pieces in ten (config 1: 28.6 against
    // 26.5 us), because the bytes a staging kernel keeps in flight are bounded by shared memory (about 19 MB over
    // the whole GPU) and that is just the latency-bandwidth product of HBM, while the gather kernel has every
    // load of the launch in flight at once.  GRASS_TUNE_COMPRESS_ROWS = 1 selects it.
    if (grass::tuning(GRASS_TUNE_COMPRESS_ROWS, 0) == 1 &&
        grass::compress_rows_fits(g, dt == GRASS_F32 ? 4 : 2, p, ld, idx, kprime, spec->k, n))
        return grass::launch_compress_rows(g, dt, n, p, ld, idx, kprime, *spec, out, ld_out, dev_status, st, out_bf16);
    if (dt == GRASS_F32)
        return grass::dispatch_compress<float>((const float*)g, n, p, ld, idx, kprime, *spec, out, ld_out,
                                               dev_status, st, out_bf16);
    return grass::dispatch_compress<__nv_bfloat16>((const __nv_bfloat16*)g, n, p, ld, idx, kprime, *spec, out,
                                                   ld_out, dev_status, st, out_bf16);
}

extern "C" grass_status grass_compress(const void* g, grass_dtype dt, int64_t n, int64_t p, int64_t ld,
                                       const uint32_t* idx, int64_t kprime, const grass_sjlt_spec* spec,
                                       float* out, int64_t ld_out, uint32_t* dev_status, void* stream)
{
    return grass_compress_out(g, dt, n, p, ld, idx, kprime, spec, out, GRASS_F32, ld_out, dev_status, stream);
}
