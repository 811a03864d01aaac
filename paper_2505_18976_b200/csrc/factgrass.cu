// factgrass_compress: FactGraSS for linear layers (Section 3.3.2) as one fused kernel.
//
//   stage 1 (sparsification)  gather A[b,t,mask_in], G[b,t,mask_out] straight from HBM; every thread owns
//                             one masked column and writes 8 consecutive tokens of it as one 16-byte chunk
//                             of a K-major, 64-byte-swizzled tensor-core operand tile in shared memory;
//   stage 2 (reconstruction)  C[a,c] += sum_t a'_t[a] * b'_t[c]   (Eq. 2 with selection matrices)
//                             with tcgen05.mma, bf16 in / fp32 accumulate in tensor memory, tokens =
//                             contraction dim; fp32 factors as three exact bf16 pieces and six products;
//   stage 3 (sparse proj.)    every accumulator entry q = a*kout + c is hashed from the seed and
//                             added into a k-bin accumulator in shared memory, which is flushed to
//                             the output row with coalesced reductions.
//
// A work item is (layer, sample, token chunk, block tile).  The token sum is split over chunks
// because SJLT is linear: partial blocks are projected separately and their projections add up in
// the output row.  Neither the masked factors nor the k'_in x k'_out block ever reach HBM.
#include "factgrass_common.cuh"

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

namespace grass {

// What happens to the finished k'_in x k'_out block.
constexpr int kEpiSjlt = 0;   // FactGraSS stage 3: hash every entry into the k-bin accumulator
constexpr int kEpiBlock = 2;  // factorised Mask alone (Section 3.2): add the block itself into out[b, off + a*kout + c]
constexpr int kEpiRaw = 1;    // add scale * block into a dense symmetric matrix (projected FIM, see grass_fim.cu):
                              // only tiles on or above the diagonal are computed, the others are mirrored

// TM x TN block tile of C per CTA (TM = MMA M: masked input coordinates, TN = MMA N: masked output
// coordinates, contraction over tokens).  F32: fp32 inputs, split exactly into three bf16 pieces.
// A NULL mask means the identity (coordinate = position).
template <int TM, int TN, bool F32, int EPI>
__global__ void __launch_bounds__(kFgThreads)
factgrass_kernel(const LayerDesc* __restrict__ descs, const __grid_constant__ LayerDesc single, int32_t B,
                 int32_t T, const int64_t* __restrict__ tok_begin, const int32_t* __restrict__ tok_count,
                 int32_t max_tiles, int32_t chunk_len, float* __restrict__ out, int64_t ld_out,
                 uint32_t* dev_status, int nprod, int flush_mode)
{
    using elem_t = typename in_elem<F32>::type;
    constexpr int NP = F32 ? 3 : 1;                       // bf16 pieces per operand
    constexpr int A_TILE = TM * (int)tc::ROW_BYTES;       // one piece of the A operand tile (TM rows x 32 tokens)
    constexpr int G_TILE = TN * (int)tc::ROW_BYTES;
    constexpr int STAGE = NP * (A_TILE + G_TILE);
    constexpr int NBUF = kFgBufs;
    constexpr int GA = kFgThreads / TM, GG = kFgThreads / TN;   // 8-token groups covered by one pass
    constexpr int PASS_A = 4 / GA, PASS_G = 4 / GG;             // passes per 32-token stage
    constexpr uint32_t ACC_COLS = F32 ? 2 * TN : TN;            // fp32 accumulator columns in tensor memory
    static_assert((TM == 64 || TM == 128) && (TN == 64 || TN == 128), "tile");
    static_assert(STAGE % 512 == 0, "operand tiles stay 512-byte aligned");

    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[NBUF + 1];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    float* bins = reinterpret_cast<float*>(smem + NBUF * STAGE);

    const LayerDesc& L = descs ? descs[blockIdx.z] : single;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.y;
    // block tiles of one token chunk are neighbours in launch order: the rows they share are read from
    // HBM once and from L2 by the others
    const int chunk = blockIdx.x / max_tiles;
    const int tile = blockIdx.x % max_tiles;
    // a layer with an empty factor mask has no block at all (its output range stays zero): leave before
    // any division by its tile counts, any mask load or any allocation
    if (L.tiles_m <= 0 || L.tiles_n <= 0) return;
    const int tm = tile % L.tiles_m, tn = tile / L.tiles_m;
    if (tn >= L.tiles_n) return;
    if (EPI == kEpiRaw && tn < tm) return;
    const int kin = L.kin, kout = L.kout;
    const int64_t d_in = L.d_in, d_out = L.d_out;
    const uint32_t k = L.k;
    const uint32_t s = L.s;
    const uint64_t seed = L.seed;
    // this sample's tokens: rows [row0, row0 + Tb) of A and G (Tb = T and row0 = b*T without the
    // per-sample arrays); a length outside [0, T] is clamped and flagged
    int Tb = T;
    if (tok_count) {
        Tb = __ldg(tok_count + b);
        if (Tb < 0 || Tb > T) {
            if (dev_status && threadIdx.x == 0 && blockIdx.x == 0) atomicOr(dev_status, GRASS_DEV_BAD_LENGTH);
            Tb = Tb < 0 ? 0 : T;
        }
    }
    const int64_t row0 = tok_begin ? __ldg(tok_begin + b) : (int64_t)b * T;
    const int t_begin = chunk * chunk_len;
    const int t_end = min(Tb, t_begin + chunk_len);
    if (t_begin >= t_end) return;          // whole CTA leaves together, before any barrier or allocation
    const bool smem_bins = EPI == kEpiSjlt && L.use_smem_bins != 0;

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
    if (smem_bins)
        for (uint32_t i = tid; i < k; i += kFgThreads) bins[i] = 0.0f;
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_slot;

    // this thread's gather columns (fixed for the whole chunk): masked coordinate aL of the A tile and
    // gL of the G tile; per pass it reads 8 consecutive tokens of them (one 16-byte operand chunk)
    bool bad = false;
    const int aL = tid % TM, gL = tid % TN;
    const int grpA = tid / TM, grpG = tid / TN;
    bool okA = tm * TM + aL < kin, okG = tn * TN + gL < kout;
    uint32_t colA = okA ? (L.mask_in ? __ldg(L.mask_in + tm * TM + aL) : (uint32_t)(tm * TM + aL)) : 0u;
    uint32_t colG = okG ? (L.mask_out ? __ldg(L.mask_out + tn * TN + gL) : (uint32_t)(tn * TN + gL)) : 0u;
    if (okA && colA >= (uint32_t)L.d_in) { bad = true; okA = false; colA = 0; }
    if (okG && colG >= (uint32_t)L.d_out) { bad = true; okG = false; colG = 0; }
    const elem_t* pA = reinterpret_cast<const elem_t*>(L.A) + row0 * d_in + colA;
    const elem_t* pG = reinterpret_cast<const elem_t*>(L.G) + row0 * d_out + colG;

    uint32_t ra[PASS_A][8], rg[PASS_G][8];   // gathered elements: fp32 bits, or bf16 bits in the low half
    auto load1 = [](const elem_t* p) -> uint32_t {
        if constexpr (F32) return gather_u32(p); else return (uint32_t)gather_u16(p);
    };
    auto prefetch = [&](int t0) {
#pragma unroll
        for (int ps = 0; ps < PASS_A; ++ps)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int t = t0 + (ps * GA + grpA) * 8 + i;
                ra[ps][i] = (okA && t < t_end) ? load1(pA + (int64_t)t * d_in) : 0u;
            }
#pragma unroll
        for (int ps = 0; ps < PASS_G; ++ps)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int t = t0 + (ps * GG + grpG) * 8 + i;
                rg[ps][i] = (okG && t < t_end) ? load1(pG + (int64_t)t * d_out) : 0u;
            }
    };
    // registers -> operand tiles of stage `buf`: row = masked coordinate, 16-byte chunk = 8-token group
    auto put = [&](unsigned char* tile0, int piece_bytes, int row, int ch, const uint32_t (&v)[8]) {
        const uint32_t off = tc::operand_chunk_offset(row, ch);
        if constexpr (F32) {
            float x[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = __uint_as_float(v[i]);
            uint4 hi, mid, lo;
            tc::split8(x, hi, mid, lo);
            *reinterpret_cast<uint4*>(tile0 + off) = hi;
            *reinterpret_cast<uint4*>(tile0 + piece_bytes + off) = mid;
            *reinterpret_cast<uint4*>(tile0 + 2 * piece_bytes + off) = lo;
        } else {
            *reinterpret_cast<uint4*>(tile0 + off) = pack8_bf16(v);
        }
    };
    auto stash = [&](int buf) {
        unsigned char* sa = smem + buf * STAGE;
        unsigned char* sg = sa + NP * A_TILE;
#pragma unroll
        for (int ps = 0; ps < PASS_A; ++ps) put(sa, A_TILE, aL, ps * GA + grpA, ra[ps]);
#pragma unroll
        for (int ps = 0; ps < PASS_G; ++ps) put(sg, G_TILE, gL, ps * GG + grpG, rg[ps]);
    };

    const uint32_t smem_base = tc::smem_u32(smem);
    const uint32_t idesc = tc::make_idesc(TM, TN);
    bool ok = true;
    prefetch(t_begin);
    int it = 0;
    for (int t0 = t_begin; t0 < t_end; t0 += kTokTile, ++it) {
        const int buf = it % NBUF;
        // the MMAs that read this buffer two steps ago must have finished before it is overwritten
        if (it >= NBUF) ok = tc::mbar_wait(bar0 + 8 * buf, (uint32_t)(it / NBUF - 1) & 1u) && ok;
        stash(buf);
        if (t0 + kTokTile < t_end) prefetch(t0 + kTokTile);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_base + buf * STAGE, g0 = a0 + NP * A_TILE;
#pragma unroll
            for (int ks = 0; ks < kTokTile / 16; ++ks) {
                if constexpr (F32) {
                    // hi*hi goes to the first accumulator, the correction terms to the second (the tensor core
                    // truncates after every accumulation, so the large sum sees as few of them as possible)
#pragma unroll
                    for (int q = 0; q < 6; ++q) {
                        if (q >= nprod) break;
                        const uint64_t ad = tc::make_smem_desc(a0 + tc::split_piece_a(q) * A_TILE + ks * 32);
                        const uint64_t gd = tc::make_smem_desc(g0 + tc::split_piece_b(q) * G_TILE + ks * 32);
                        tc::umma_bf16(q == 0 ? tmem_d : tmem_d + TN, ad, gd, idesc, (it > 0 || ks > 0 || q > 1) ? 1u : 0u);
                    }
                } else {
                    tc::umma_bf16(tmem_d, tc::make_smem_desc(a0 + ks * 32), tc::make_smem_desc(g0 + ks * 32), idesc,
                                  (it > 0 || ks > 0) ? 1u : 0u);
                }
            }
            tc::umma_commit(bar0 + 8 * buf);                       // buffer free once these MMAs have read it
            if (t0 + kTokTile >= t_end) tc::umma_commit(bar_done); // accumulator complete
        }
    }
    if (bad && dev_status) atomicOr(dev_status, GRASS_DEV_BAD_INDEX);
    ok = tc::mbar_wait(bar_done, 0) && ok;
    if (!ok) abort_flag = 1;
    __syncthreads();
    ok = abort_flag == 0;
    if (!ok && tid == 0 && dev_status) atomicOr(dev_status, GRASS_DEV_TIMEOUT);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    // stage 3: SJLT of the block; flat position q = a*kout + c (input-major flattening).
    // Accumulator row a sits in tensor-memory lane a (TM = 128) or lane (a % 16) + 32 * (a / 16) (TM = 64);
    // warp w may read lanes 32 * (w % 4) .. + 31; the two warps that share a lane quarter split the columns.
    float* orow = out + (int64_t)b * ld_out + L.out_offset;
    const float scale = 1.0f / sqrtf((float)s);
    const int quarter = warp & 3;
    const uint32_t tq = tmem_d + ((uint32_t)(quarter * 32) << 16);
    auto project = [&](int a, int c, float val) {
        if constexpr (EPI == kEpiBlock) {
            if (a < kin && c < kout && val != 0.0f) atomicAdd(orow + (int64_t)a * kout + c, val);
        } else if constexpr (EPI == kEpiRaw) {
            // tiles above the diagonal fill their mirror image too; a diagonal tile uses its upper half
            if (a < kin && c < kout && (tm != tn || a <= c)) {
                const float sv = val * L.scale;
                atomicAdd(out + (int64_t)a * ld_out + c, sv);
                if (a != c) atomicAdd(out + (int64_t)c * ld_out + a, sv);
            }
        } else if (a < kin && c < kout && val != 0.0f) {
            const uint64_t q = (uint64_t)a * (uint64_t)kout + (uint64_t)c;
            for (uint32_t r = 0; r < s; ++r) {
                const uint64_t h = sjlt_hash_counter(seed, q * s + r + 1);
                const uint32_t bk = sjlt_bucket(h, k);
                const float sv = (s == 1) ? sjlt_signed(h, val) : sjlt_signed(h, val) * scale;
                if (smem_bins) atomicAdd(&bins[bk], sv);
                else atomicAdd(orow + bk, sv);
            }
        }
    };
    if (ok) {
        if constexpr (TM == 64) {
            // 16 rows x 32 columns per warp, 16 values per thread
            const int c0 = (warp >> 2) * 32;
            uint32_t v[16];
            tc::tmem_ld_16x256b_x4(tq + (uint32_t)c0, v);
            if constexpr (F32) {
                uint32_t w[16];
                tc::tmem_ld_16x256b_x4(tq + (uint32_t)(TN + c0), w);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) + __uint_as_float(w[e]));
            } else {
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            }
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int a = tm * TM + quarter * 16 + (lane >> 2) + 8 * ((e & 3) >> 1);
                const int c = tn * TN + c0 + 8 * (e >> 2) + 2 * (lane & 3) + (e & 1);
                project(a, c, __uint_as_float(v[e]));
            }
        } else {
            const int a = tm * TM + quarter * 32 + lane;
#pragma unroll 1
            for (int c0 = (warp >> 2) * 32; c0 < TN; c0 += 64) {
                uint32_t v[32];
                tc::tmem_ld32(tq + (uint32_t)c0, v);
                if constexpr (F32) {
                    uint32_t w[32];
                    tc::tmem_ld32(tq + (uint32_t)(TN + c0), w);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) + __uint_as_float(w[e]));
                } else {
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                }
#pragma unroll
                for (int e = 0; e < 32; ++e) project(a, tn * TN + c0 + e, __uint_as_float(v[e]));
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(ACC_COLS) : "memory");
    }
    // flush_mode 0: several thread blocks feed the row: reductions into the zeroed row.  1 / 2: this thread block is
    // the only one of its (layer, sample), so the bins ARE the row: plain stores, fp32 or bf16 (rounded here, once)
    if (smem_bins && flush_mode != 0) {
        for (uint32_t i = tid; i < k; i += kFgThreads)
            store_out(out, (int64_t)b * ld_out + L.out_offset + i, bins[i], flush_mode == 2);
    } else if (smem_bins && ok) {
        for (uint32_t i = tid; i < k; i += kFgThreads) {
            const float v = bins[i];
            if (v != 0.0f) atomicAdd(orow + i, v);
        }
    }
}

// zeroes every layer's [out_offset, out_offset + k) range of every sample row
__global__ void factgrass_zero_kernel(const LayerDesc* __restrict__ descs, const __grid_constant__ LayerDesc single,
                                      float* __restrict__ out, int64_t ld_out, int out_bf16)
{
    const LayerDesc& L = descs ? descs[blockIdx.z] : single;
    const int64_t orow = (int64_t)blockIdx.y * ld_out + L.out_offset;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < L.k; i += gridDim.x * blockDim.x)
        store_out(out, orow + i, 0.0f, out_bf16);
}

static grass_status fill_desc(LayerDesc& d, const factgrass_layer& l, int tile, int32_t T)
{
    if (l.spec.k == 0 || l.spec.s == 0) return GRASS_ERR_INVALID_ARG;
    if (l.d_in <= 0 || l.d_out <= 0 || l.kin < 0 || l.kout < 0 || l.kin > l.d_in || l.kout > l.d_out)
        return GRASS_ERR_INVALID_ARG;
    if (l.out_offset < 0) return GRASS_ERR_INVALID_ARG;
    if ((l.kin > 0 && l.kout > 0 && T > 0) && (!l.A || !l.G)) return GRASS_ERR_INVALID_ARG;
    // a NULL mask is the identity; an empty mask (k' = 0) needs no list either
    if ((!l.mask_in && l.kin != l.d_in && l.kin != 0) || (!l.mask_out && l.kout != l.d_out && l.kout != 0))
        return GRASS_ERR_INVALID_ARG;
    d.A = l.A;
    d.G = l.G;
    d.mask_in = l.mask_in;
    d.mask_out = l.mask_out;
    d.d_in = l.d_in;
    d.d_out = l.d_out;
    d.kin = l.kin;
    d.kout = l.kout;
    d.k = l.spec.k;
    d.s = l.spec.s;
    d.seed = l.spec.seed;
    d.out_offset = l.out_offset;
    d.tiles_m = (l.kin + tile - 1) / tile;
    d.tiles_n = (l.kout + tile - 1) / tile;
    d.use_smem_bins = (size_t)l.spec.k * sizeof(float) <= kMaxSmemBins;
    d.scale = 1.0f;
    return GRASS_OK;
}

static grass_status run_factgrass(const factgrass_layer* layers, int32_t L, grass_dtype dt, int32_t B, int32_t T,
                                  const int64_t* tok_begin, const int32_t* tok_count, float* out, int64_t ld_out,
                                  void* workspace, size_t workspace_bytes, uint32_t* dev_status, cudaStream_t st,
                                  int epi = kEpiSjlt, int out_bf16 = 0)
{
    if (L < 0 || B < 0 || T < 0 || (L > 0 && !layers)) return GRASS_ERR_INVALID_ARG;
    if (dt != GRASS_BF16 && dt != GRASS_F32) return GRASS_ERR_INVALID_ARG;
    if (L == 0 || B == 0) return GRASS_OK;
    if (!out) return GRASS_ERR_INVALID_ARG;
    if (L > 65535 || B > 65535) return GRASS_ERR_UNSUPPORTED;

    int max_kk = 0;
    uint32_t max_k = 0, max_k_smem = 0;
    for (int l = 0; l < L; ++l) {
        if ((size_t)layers[l].spec.k * sizeof(float) <= kMaxSmemBins && layers[l].spec.k > max_k_smem)
            max_k_smem = layers[l].spec.k;
        if (layers[l].kin > max_kk) max_kk = layers[l].kin;
        if (layers[l].kout > max_kk) max_kk = layers[l].kout;
        if (layers[l].spec.k > max_k) max_k = layers[l].spec.k;
        if (layers[l].out_offset < 0 || layers[l].out_offset + (int64_t)layers[l].spec.k > ld_out)
            return GRASS_ERR_INVALID_ARG;
    }
    // 64 x 64 block tiles; larger blocks are covered by several tiles whose shared rows come from L2.
    // The 128 x 128 variant serves the projected FIM and comparison runs (GRASS_TUNE_FACTGRASS_TILE = 128).
    const int tile = tuning(GRASS_TUNE_FACTGRASS_TILE, 64) == 128 && max_kk > 64 ? 128 : 64;

    if (!workspace && L != 1) return GRASS_ERR_INVALID_ARG;
    if (workspace && (workspace_bytes < (size_t)L * sizeof(LayerDesc) || ((uintptr_t)workspace & 15)))
        return GRASS_ERR_INVALID_ARG;
    // every layer is checked on the host before anything touches the device
    for (int l = 0; l < L; ++l) {
        LayerDesc probe;
        const grass_status rc = fill_desc(probe, layers[l], tile, T);
        if (rc != GRASS_OK) return rc;
    }
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return GRASS_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GRASS_ERR_CUDA;
    const bool f32 = dt == GRASS_F32;

    // Launches of about one wave (few layers x samples, bf16 factors, blocks of one tile) take the cluster kernel:
    // one cluster per (layer, sample), no zero-fill, no global reductions (factgrass_cluster.cu).
    ClusterPlan cplan;
    int cluster_nc = 0, cluster_chunk = 0;
    auto plan_cluster = [&](const LayerDesc* hd) {
        if (epi != kEpiSjlt || f32 || T <= 0) return;
        const int64_t forced = tuning(GRASS_TUNE_FACTGRASS_PATH, -1);
        if (forced == 0 || !cluster_path_fits(hd, L, &cplan)) return;
        const int64_t items = (int64_t)L * B, slots = (int64_t)sms * cplan.per_sm;
        if (items > slots && forced != 1) return;
        // clusters of 1, 2, 4 or 8 thread blocks: as many as fill the machine, each with at least two 32-token steps;
        // no accumulator runs over more than 8,192 tokens
        auto pow2_floor = [](int64_t v) { int64_t p = 1; while (p * 2 <= v) p *= 2; return p; };
        int64_t nc = pow2_floor(std::max<int64_t>(1, std::min<int64_t>(8, slots / std::max<int64_t>(items, 1))));
        nc = std::min<int64_t>(nc, pow2_floor(std::max<int64_t>(1, T / (2 * kTokTile))));
        int64_t chunk = ((T + nc - 1) / nc + kTokTile - 1) / kTokTile * kTokTile;
        const int64_t forced_chunk = tuning(GRASS_TUNE_FACTGRASS_CHUNK, -1);
        if (forced_chunk > 0) {
            chunk = std::max<int64_t>(kTokTile, (forced_chunk + kTokTile - 1) / kTokTile * kTokTile);
            const int64_t need = (T + chunk - 1) / chunk;
            nc = 1;
            while (nc < need) nc *= 2;
        }
        if (nc > 8 || chunk > 8192) return;
        cluster_nc = (int)nc;
        cluster_chunk = (int)chunk;
    };

    // a single layer travels as a kernel parameter: no descriptor copy, whoever provided a workspace
    const bool grouped = workspace != nullptr && L > 1;
    LayerDesc single;
    std::memset(&single, 0, sizeof single);
    LayerDesc* dev_descs = nullptr;
    int max_tiles = 1;
    if (grouped) {
        // descriptors are staged on the host stack / heap and copied on the stream
        LayerDesc stack_buf[256];
        LayerDesc* host = L <= 256 ? stack_buf : (LayerDesc*)std::malloc((size_t)L * sizeof(LayerDesc));
        if (!host) return GRASS_ERR_CUDA;
        grass_status rc = GRASS_OK;
        for (int l = 0; l < L && rc == GRASS_OK; ++l) {
            rc = fill_desc(host[l], layers[l], tile, T);
            if (rc == GRASS_OK && host[l].tiles_m * host[l].tiles_n > max_tiles)
                max_tiles = host[l].tiles_m * host[l].tiles_n;
        }
        if (rc == GRASS_OK) plan_cluster(host);
        if (rc == GRASS_OK)
            rc = cuda_ok(cudaMemcpyAsync(workspace, host, (size_t)L * sizeof(LayerDesc), cudaMemcpyHostToDevice, st));
        if (host != stack_buf) std::free(host);
        if (rc != GRASS_OK) return rc;
        dev_descs = (LayerDesc*)workspace;
    } else {
        grass_status rc = fill_desc(single, layers[0], tile, T);
        if (rc != GRASS_OK) return rc;
        max_tiles = single.tiles_m * single.tiles_n;
        plan_cluster(&single);
    }
    if (cluster_nc > 0)
        return launch_factgrass_cluster(dev_descs, single, cplan, L, B, T, tok_begin, tok_count, cluster_nc,
                                        cluster_chunk, out, ld_out, dev_status, st, out_bf16);
    // A bf16 row is rounded once, at the final store, so the streaming kernel takes it only where one thread block
    // owns a whole (layer, sample): one block tile, the whole token sum (at most 8,192 tokens), bins in shared memory
    if (out_bf16 && (max_tiles > 1 || max_k != max_k_smem || T > 8192 || epi != kEpiSjlt)) return GRASS_ERR_UNSUPPORTED;

    // zero the output ranges (the compress kernel accumulates partial projections into them)
    {
        dim3 zg((max_k + 1023) / 1024 > 0 ? (max_k + 1023) / 1024 : 1, (unsigned)B, (unsigned)L);
        if (zg.x > 64) zg.x = 64;
        factgrass_zero_kernel<<<zg, 256, 0, st>>>(dev_descs, single, out, ld_out, out_bf16);
        if (launch_status() != GRASS_OK) return GRASS_ERR_CUDA;
    }
    if (T == 0 || max_tiles == 0) return GRASS_OK;

    const size_t bins_bytes = epi == kEpiSjlt ? (size_t)max_k_smem * sizeof(float) : 0;
    auto launch = [&](auto kern, size_t stage_bytes) -> grass_status {
        const size_t smem = kFgBufs * stage_bytes + bins_bytes;
        // static shared memory counts toward the 48 KB default limit too
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return GRASS_ERR_CUDA;
        cudaFuncAttributes fa;
        if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) return GRASS_ERR_CUDA;
        const size_t cta_smem = smem + fa.sharedSizeBytes + 1024;   // + the per-CTA reservation
        // resident CTAs per SM from the kernel's own footprint: registers, threads, tensor-memory columns
        // (which the runtime's occupancy query does not count) and shared memory
        auto resident = [&](size_t smem_per_sm) {
            int r = 65536 / (fa.numRegs > 0 ? fa.numRegs * kFgThreads : 65536);
            r = std::min(r, 2048 / kFgThreads);
            r = std::min(r, 512 / (tile * (f32 ? 2 : 1)));
            r = std::min(r, (int)(smem_per_sm / cta_smem));
            return r < 1 ? 1 : r;
        };
        const int64_t base_items = (int64_t)L * B * max_tiles;
        // Gathered loads are tracked in L1 while in flight, and L1 is what the shared-memory carve-out leaves
        // of the SM's 256 KB.  A launch of several waves (the HBM-streaming regime) runs fastest with one to
        // three resident CTAs and a 64 KB carve-out; a launch of about one wave wants more CTA slots but still
        // keeps about 90 KB of L1 (carve-out at most 164 KB).  The driver's default would size the carve-out
        // for the largest number of CTAs and starve L1.
        const bool streaming = base_items >= 2 * (int64_t)sms * resident(std::max<size_t>(64 * 1024, cta_smem));
        const size_t cap = std::max<size_t>((streaming ? 64 : 164) * 1024, cta_smem);
        int per_sm = resident(cap);
        int carve = 100;
        {
            const int configs_kb[] = {8, 16, 32, 64, 100, 132, 164, 196, 228};
            for (int kb : configs_kb)
                if ((size_t)kb * 1024 >= (size_t)per_sm * cta_smem) { carve = kb * 100 / 228; break; }
        }
        carve = (int)tuning(GRASS_TUNE_FACTGRASS_CARVEOUT, carve);
        if (cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, carve) != cudaSuccess)
            return GRASS_ERR_CUDA;
        // token chunks.  Every chunk pays a fixed projection epilogue (tile*tile hashes and a k-bin flush),
        // so chunks are as long as the machine allows: when there are fewer work items than resident CTA
        // slots the token sum is split just enough to fill one wave; otherwise just enough for ~8 waves
        // so that the last, partial wave costs little.
        const int64_t slots = (int64_t)sms * per_sm;
        const int min_chunk = 64;
        int64_t want = base_items < slots ? slots / base_items : (8 * slots + base_items - 1) / base_items;
        int64_t max_chunks = (T + min_chunk - 1) / min_chunk;
        // the tensor core truncates its fp32 accumulator after every MMA: no accumulator runs over more than
        // 8,192 tokens, so that this bias stays near 1e-5 of the result however long the sequence is
        want = std::max<int64_t>(want, ((int64_t)T + 8191) / 8192);
        if (want > max_chunks) want = max_chunks;
        if (want < 1) want = 1;
        int chunk_len = (int)((T + want - 1) / want);
        chunk_len = (chunk_len + kTokTile - 1) / kTokTile * kTokTile;
        chunk_len = (int)tuning(GRASS_TUNE_FACTGRASS_CHUNK, chunk_len);
        if (out_bf16) chunk_len = T;
        if (chunk_len < kTokTile) chunk_len = kTokTile;
        chunk_len = (chunk_len + kTokTile - 1) / kTokTile * kTokTile;
        const int nchunks = (T + chunk_len - 1) / chunk_len;
        dim3 grid((unsigned)(nchunks * max_tiles), (unsigned)B, (unsigned)L);
        int nprod = (int)tuning(GRASS_TUNE_SPLIT_PRODUCTS, tc::kSplitProductsDefault);
        if (nprod != 3 && nprod != 4) nprod = 6;
        kern<<<grid, kFgThreads, smem, st>>>(dev_descs, single, B, T, tok_begin, tok_count, max_tiles, chunk_len, out,
                                             ld_out, dev_status, nprod, out_bf16 ? 2 : 0);
        return launch_status();
    };
    const size_t piece = (size_t)tile * tc::ROW_BYTES * 2;   // one bf16 piece of the A tile plus one of the G tile
    if (epi == kEpiBlock) {
        if (tile == 64)
            return f32 ? launch(factgrass_kernel<64, 64, true, kEpiBlock>, 3 * piece)
                       : launch(factgrass_kernel<64, 64, false, kEpiBlock>, piece);
        return f32 ? launch(factgrass_kernel<128, 128, true, kEpiBlock>, 3 * piece)
                   : launch(factgrass_kernel<128, 128, false, kEpiBlock>, piece);
    }
    if (tile == 64)
        return f32 ? launch(factgrass_kernel<64, 64, true, kEpiSjlt>, 3 * piece)
                   : launch(factgrass_kernel<64, 64, false, kEpiSjlt>, piece);
    return f32 ? launch(factgrass_kernel<128, 128, true, kEpiSjlt>, 3 * piece)
               : launch(factgrass_kernel<128, 128, false, kEpiSjlt>, piece);
}

// Factorised Mask without projection: the layers' specs are replaced by k = kin * kout (the block itself
// is the output) and the kernels run with the block epilogue.
static grass_status run_factmask(const factgrass_layer* layers, int32_t L, grass_dtype dt, int32_t B, int32_t T,
                                 float* out, int64_t ld_out, void* workspace, size_t workspace_bytes,
                                 uint32_t* dev_status, cudaStream_t st)
{
    if (L < 0 || (L > 0 && !layers)) return GRASS_ERR_INVALID_ARG;
    std::vector<factgrass_layer> tmp(layers, layers + L);
    for (auto& l : tmp) {
        if (l.kin < 0 || l.kout < 0 || (int64_t)l.kin * l.kout > 0x7FFFFFFFLL) return GRASS_ERR_INVALID_ARG;
        l.spec.k = (uint32_t)std::max<int64_t>((int64_t)l.kin * l.kout, 1);
        l.spec.s = 1;
        l.spec.seed = 0;
    }
    return run_factgrass(tmp.data(), L, dt, B, T, nullptr, nullptr, out, ld_out, workspace, workspace_bytes, dev_status,
                         st, kEpiBlock);
}

// Projected Fisher information matrix F = scale * X^T X of the n rows of X (n x k fp32, row stride ld):
// the Kronecker-sum contraction of the FactGraSS kernel with both factors = X, identity masks and the
// raw-block epilogue.  F (k x k, row stride ld_f) must have been zeroed on the stream.
grass_status launch_fim(const float* X, int64_t n, int64_t k, int64_t ld, float scale, float* F, int64_t ld_f,
                        cudaStream_t st)
{
    constexpr int tile = 128;
    LayerDesc d;
    std::memset(&d, 0, sizeof d);
    d.A = X;
    d.G = X;
    d.d_in = d.d_out = (int32_t)ld;
    d.kin = d.kout = (int32_t)k;
    d.tiles_m = d.tiles_n = (int32_t)((k + tile - 1) / tile);
    d.scale = scale;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return GRASS_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GRASS_ERR_CUDA;
    auto kern = factgrass_kernel<tile, tile, true, kEpiRaw>;
    const size_t smem = kFgBufs * 3 * (size_t)tile * tc::ROW_BYTES * 2;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return GRASS_ERR_CUDA;
    const int per_sm = 2;   // 97 KB of shared memory and 256 tensor-memory columns per CTA; 196 KB carve-out
    if (cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 85) != cudaSuccess)
        return GRASS_ERR_CUDA;
    // sample chunks: enough CTAs for ~4 waves of the tiles on or above the diagonal, at least 256 samples each
    const int64_t tiles = (int64_t)d.tiles_m * (d.tiles_m + 1) / 2;
    int64_t want = (4 * (int64_t)sms * per_sm + tiles - 1) / tiles;
    const int64_t max_chunks = (n + 255) / 256;
    want = std::max<int64_t>(want, (n + 8191) / 8192);   // bounded accumulation runs, as for the token chunks
    if (want > max_chunks) want = max_chunks;
    if (want < 1) want = 1;
    int64_t chunk_len = (n + want - 1) / want;
    chunk_len = (chunk_len + kTokTile - 1) / kTokTile * kTokTile;
    const int64_t nchunks = (n + chunk_len - 1) / chunk_len;
    const int64_t gx = nchunks * d.tiles_m * d.tiles_n;
    if (gx > 0x7FFFFFFFLL || chunk_len > 0x7FFFFFFFLL) return GRASS_ERR_UNSUPPORTED;
    dim3 grid((unsigned)gx, 1, 1);
    int nprod = (int)tuning(GRASS_TUNE_SPLIT_PRODUCTS, tc::kSplitProductsDefault);
    if (nprod != 3 && nprod != 4) nprod = 6;
    kern<<<grid, kFgThreads, smem, st>>>(nullptr, d, 1, (int32_t)n, nullptr, nullptr, d.tiles_m * d.tiles_n,
                                         (int32_t)chunk_len, F, ld_f, nullptr, nprod, 0);
    return launch_status();
}

}  // namespace grass

extern "C" grass_status factgrass_compress(const void* A, const void* G, grass_dtype dt, int32_t B, int32_t T,
                                           int32_t d_in, int32_t d_out, const uint32_t* mask_in, int32_t kin,
                                           const uint32_t* mask_out, int32_t kout, const grass_sjlt_spec* spec,
                                           float* out, int64_t ld_out, uint32_t* dev_status, void* stream)
{
    if (!spec) return GRASS_ERR_INVALID_ARG;
    factgrass_layer l;
    l.A = A;
    l.G = G;
    l.mask_in = mask_in;
    l.mask_out = mask_out;
    l.d_in = d_in;
    l.d_out = d_out;
    l.kin = kin;
    l.kout = kout;
    l.spec = *spec;
    l.out_offset = 0;
    return grass::run_factgrass(&l, 1, dt, B, T, nullptr, nullptr, out, ld_out, nullptr, 0, dev_status,
                                (cudaStream_t)stream);
}

extern "C" grass_status factgrass_compress_varlen(const void* A, const void* G, grass_dtype dt, int32_t B,
                                                  int32_t T_max, const int64_t* tok_begin, const int32_t* tok_count,
                                                  int32_t d_in, int32_t d_out, const uint32_t* mask_in, int32_t kin,
                                                  const uint32_t* mask_out, int32_t kout, const grass_sjlt_spec* spec,
                                                  float* out, int64_t ld_out, uint32_t* dev_status, void* stream)
{
    if (!spec) return GRASS_ERR_INVALID_ARG;
    factgrass_layer l;
    l.A = A;
    l.G = G;
    l.mask_in = mask_in;
    l.mask_out = mask_out;
    l.d_in = d_in;
    l.d_out = d_out;
    l.kin = kin;
    l.kout = kout;
    l.spec = *spec;
    l.out_offset = 0;
    return grass::run_factgrass(&l, 1, dt, B, T_max, tok_begin, tok_count, out, ld_out, nullptr, 0, dev_status,
                                (cudaStream_t)stream);
}

extern "C" grass_status factmask_compress(const void* A, const void* G, grass_dtype dt, int32_t B, int32_t T,
                                          int32_t d_in, int32_t d_out, const uint32_t* mask_in, int32_t kin,
                                          const uint32_t* mask_out, int32_t kout, float* out, int64_t ld_out,
                                          uint32_t* dev_status, void* stream)
{
    factgrass_layer l;
    l.A = A;
    l.G = G;
    l.mask_in = mask_in;
    l.mask_out = mask_out;
    l.d_in = d_in;
    l.d_out = d_out;
    l.kin = kin;
    l.kout = kout;
    l.spec.k = 1;
    l.spec.s = 1;
    l.spec.seed = 0;
    l.out_offset = 0;
    return grass::run_factmask(&l, 1, dt, B, T, out, ld_out, nullptr, 0, dev_status, (cudaStream_t)stream);
}

extern "C" grass_status factmask_compress_grouped(const factgrass_layer* layers, int32_t L, grass_dtype dt, int32_t B,
                                                  int32_t T, float* out, int64_t ld_out, void* workspace,
                                                  size_t workspace_bytes, uint32_t* dev_status, void* stream)
{
    if (!workspace) return GRASS_ERR_INVALID_ARG;
    return grass::run_factmask(layers, L, dt, B, T, out, ld_out, workspace, workspace_bytes, dev_status,
                               (cudaStream_t)stream);
}

extern "C" size_t factgrass_grouped_workspace_bytes(int32_t L)
{
    if (L <= 0) return 256;
    return ((size_t)L * sizeof(grass::LayerDesc) + 255) / 256 * 256;
}

extern "C" grass_status factgrass_compress_grouped(const factgrass_layer* layers, int32_t L, grass_dtype dt, int32_t B,
                                                   int32_t T, float* out, int64_t ld_out, void* workspace,
                                                   size_t workspace_bytes, uint32_t* dev_status, void* stream)
{
    if (!workspace) return GRASS_ERR_INVALID_ARG;
    return grass::run_factgrass(layers, L, dt, B, T, nullptr, nullptr, out, ld_out, workspace, workspace_bytes,
                                dev_status, (cudaStream_t)stream);
}

extern "C" grass_status factgrass_compress_grouped_out(const factgrass_layer* layers, int32_t L, grass_dtype dt,
                                                       int32_t B, int32_t T, void* out, grass_dtype out_dt,
                                                       int64_t ld_out, void* workspace, size_t workspace_bytes,
                                                       uint32_t* dev_status, void* stream)
{
    if (out_dt != GRASS_F32 && out_dt != GRASS_BF16) return GRASS_ERR_UNSUPPORTED;
    if (!workspace && L > 1) return GRASS_ERR_INVALID_ARG;
    return grass::run_factgrass(layers, L, dt, B, T, nullptr, nullptr, (float*)out, ld_out, workspace, workspace_bytes,
                                dev_status, (cudaStream_t)stream, grass::kEpiSjlt, out_dt == GRASS_BF16);
}

extern "C" grass_status factgrass_compress_grouped_varlen(const factgrass_layer* layers, int32_t L, grass_dtype dt,
                                                          int32_t B, int32_t T_max, const int64_t* tok_begin,
                                                          const int32_t* tok_count, float* out, int64_t ld_out,
                                                          void* workspace, size_t workspace_bytes,
                                                          uint32_t* dev_status, void* stream)
{
    if (!workspace) return GRASS_ERR_INVALID_ARG;
    return grass::run_factgrass(layers, L, dt, B, T_max, tok_begin, tok_count, out, ld_out, workspace, workspace_bytes,
                                dev_status, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// Grouped FactGraSS without a caller-provided workspace.
//
// The per-layer descriptor table of a grouped call is the only scratch memory the kernels need.
// Here it lives in a fixed array that is part of the loaded library image on every GPU, so the call
// needs no device allocation from anybody.  In host code the array's name is only a handle: the
// device address is looked up once per device with cudaGetSymbolAddress and that pointer is what
// the kernels receive.
namespace grass {

constexpr int kStaticMaxLayers = FACTGRASS_STATIC_MAX_LAYERS;
static __device__ __align__(256) unsigned char g_static_layer_table[kStaticMaxLayers * sizeof(LayerDesc)];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mutex;
static void* g_static_table_addr[kMaxDevices] = {nullptr};

// Device address of the table on the current device; resolved on first use per device.
static grass_status static_table_address(void** addr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return GRASS_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return GRASS_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_table_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_layer_table) != cudaSuccess || !p) return GRASS_ERR_CUDA;
        g_static_table_addr[dev] = p;
    }
    *addr = g_static_table_addr[dev];
    return GRASS_OK;
}

}  // namespace grass

extern "C" grass_status factgrass_compress_grouped_static(const factgrass_layer* layers, int32_t L, grass_dtype dt,
                                                          int32_t B, int32_t T, float* out, int64_t ld_out,
                                                          uint32_t* dev_status, void* stream)
{
    if (L < 0) return GRASS_ERR_INVALID_ARG;
    if (L > grass::kStaticMaxLayers) return GRASS_ERR_UNSUPPORTED;  // table holds at most 256 layers
    void* table = nullptr;
    const grass_status rc = grass::static_table_address(&table);
    if (rc != GRASS_OK) return rc;
    return grass::run_factgrass(layers, L, dt, B, T, nullptr, nullptr, out, ld_out, table,
                                (size_t)grass::kStaticMaxLayers * sizeof(grass::LayerDesc), dev_status,
                                (cudaStream_t)stream);
}
