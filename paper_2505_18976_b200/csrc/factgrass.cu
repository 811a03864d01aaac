// factgrass_compress: FactGraSS for linear layers (Section 3.3.2) as one fused kernel.
//
//   stage 1 (sparsification)  gather A[b,t,mask_in], G[b,t,mask_out] straight from HBM into
//                             token-major bf16 tiles in shared memory;
//   stage 2 (reconstruction)  C[a,c] += sum_t a'_t[a] * b'_t[c]   (Eq. 2 with selection matrices)
//                             on tensor cores, bf16 in / fp32 accumulate, tokens = contraction dim;
//   stage 3 (sparse proj.)    every accumulator entry q = a*kout + c is hashed from the seed and
//                             added into a k-bin accumulator in shared memory, which is flushed to
//                             the output row with coalesced reductions.
//
// A work item is (layer, sample, token chunk, block tile).  The token sum is split over chunks
// because SJLT is linear: partial blocks are projected separately and their projections add up in
// the output row.  Neither the masked factors nor the k'_in x k'_out block ever reach HBM.
#include "grass_common.cuh"

#include <cstdlib>
#include <cstring>
#include <mutex>

namespace grass {

constexpr int kFgThreads = 256;
constexpr int kTokTile = 32;  // tokens per pipeline stage

struct LayerDesc {
    const uint16_t* A;
    const uint16_t* G;
    const uint32_t* mask_in;
    const uint32_t* mask_out;
    int32_t d_in, d_out;
    int32_t kin, kout;
    uint32_t k, s;
    uint64_t seed;
    int64_t out_offset;
    int32_t tiles_m, tiles_n;
    int32_t use_smem_bins;
    int32_t pad_;
};
static_assert(sizeof(LayerDesc) == 88, "descriptor layout");

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                                  uint32_t smem_addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(smem_addr));
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// TM x TN block tile of C per CTA; 8 warps as 2 (rows) x 4 (cols).
template <int TM, int TN>
__global__ void __launch_bounds__(kFgThreads)
factgrass_kernel(const LayerDesc* __restrict__ descs, const __grid_constant__ LayerDesc single, int32_t B,
                 int32_t T, const int64_t* __restrict__ tok_begin, const int32_t* __restrict__ tok_count,
                 int32_t max_tiles, int32_t chunk_len, float* __restrict__ out, int64_t ld_out,
                 uint32_t* dev_status)
{
    constexpr int PA = TM * 2 + 16;  // smem row pitch in bytes (tokens x masked columns, bf16)
    constexpr int PG = TN * 2 + 16;
    constexpr int STAGE = kTokTile * (PA + PG);
    constexpr int WM = TM / 2, WN = TN / 4;
    constexpr int MT = WM / 16, NT = WN / 8;
    constexpr int RA = kTokTile * TM / kFgThreads;  // gathered A elements per thread per stage
    constexpr int RG = kTokTile * TN / kFgThreads;
    constexpr int STEP_A = kFgThreads / TM, STEP_G = kFgThreads / TN;
    static_assert(NT % 2 == 0 && MT >= 1, "warp tile");

    extern __shared__ __align__(16) unsigned char smem[];
    float* bins = reinterpret_cast<float*>(smem + 2 * STAGE);

    const LayerDesc& L = descs ? descs[blockIdx.z] : single;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.y;
    // block tiles of one token chunk are neighbours in launch order: the rows they share are read from
    // HBM once and from L2 by the others
    const int chunk = blockIdx.x / max_tiles;
    const int tile = blockIdx.x % max_tiles;
    const int tm = tile % L.tiles_m, tn = tile / L.tiles_m;
    if (tn >= L.tiles_n) return;
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
    if (t_begin >= t_end) return;
    const bool smem_bins = L.use_smem_bins != 0;

    if (smem_bins)
        for (uint32_t i = tid; i < k; i += kFgThreads) bins[i] = 0.0f;

    // this thread's gather columns (fixed for the whole chunk)
    bool bad = false;
    const int aL = tid % TM, gL = tid % TN;
    const int tokA = tid / TM, tokG = tid / TN;
    bool okA = tm * TM + aL < kin, okG = tn * TN + gL < kout;
    uint32_t colA = okA ? __ldg(L.mask_in + tm * TM + aL) : 0u;
    uint32_t colG = okG ? __ldg(L.mask_out + tn * TN + gL) : 0u;
    if (okA && colA >= (uint32_t)L.d_in) { bad = true; okA = false; colA = 0; }
    if (okG && colG >= (uint32_t)L.d_out) { bad = true; okG = false; colG = 0; }
    const uint16_t* pA = L.A + row0 * d_in + colA;
    const uint16_t* pG = L.G + row0 * d_out + colG;

    uint16_t ra[RA], rg[RG];
    auto prefetch = [&](int t0) {
#pragma unroll
        for (int i = 0; i < RA; ++i) {
            const int t = t0 + tokA + i * STEP_A;
            ra[i] = (okA && t < t_end) ? gather_u16(pA + (int64_t)t * d_in) : (uint16_t)0;
        }
#pragma unroll
        for (int i = 0; i < RG; ++i) {
            const int t = t0 + tokG + i * STEP_G;
            rg[i] = (okG && t < t_end) ? gather_u16(pG + (int64_t)t * d_out) : (uint16_t)0;
        }
    };
    auto stash = [&](int buf) {
        unsigned char* sa = smem + buf * STAGE;
        unsigned char* sg = sa + kTokTile * PA;
#pragma unroll
        for (int i = 0; i < RA; ++i)
            *reinterpret_cast<uint16_t*>(sa + (tokA + i * STEP_A) * PA + aL * 2) = ra[i];
#pragma unroll
        for (int i = 0; i < RG; ++i)
            *reinterpret_cast<uint16_t*>(sg + (tokG + i * STEP_G) * PG + gL * 2) = rg[i];
    };

    float acc[MT][NT][4];
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.0f;

    const int wm = warp >> 2, wn = warp & 3;
    const int lm = lane >> 3, lr = lane & 7;  // ldmatrix: matrix id, row within it
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);

    prefetch(t_begin);
    int buf = 0;
    for (int t0 = t_begin; t0 < t_end; t0 += kTokTile, buf ^= 1) {
        stash(buf);
        __syncthreads();
        if (t0 + kTokTile < t_end) prefetch(t0 + kTokTile);
        const uint32_t sa = smem_base + buf * STAGE;
        const uint32_t sg = sa + kTokTile * PA;
#pragma unroll
        for (int k0 = 0; k0 < kTokTile; k0 += 16) {
            uint32_t af[MT][4];
#pragma unroll
            for (int i = 0; i < MT; ++i) {
                const int row = k0 + (lm >> 1) * 8 + lr;             // token
                const int colm = wm * WM + i * 16 + (lm & 1) * 8;    // masked input coordinate
                ldmatrix_x4_trans(af[i][0], af[i][1], af[i][2], af[i][3], sa + row * PA + colm * 2);
            }
#pragma unroll
            for (int j = 0; j < NT; j += 2) {
                uint32_t b0, b1, b2, b3;
                const int row = k0 + (lm & 1) * 8 + lr;
                const int coln = wn * WN + j * 8 + (lm >> 1) * 8;
                ldmatrix_x4_trans(b0, b1, b2, b3, sg + row * PG + coln * 2);
#pragma unroll
                for (int i = 0; i < MT; ++i) {
                    mma_bf16_16816(acc[i][j], af[i], b0, b1);
                    mma_bf16_16816(acc[i][j + 1], af[i], b2, b3);
                }
            }
        }
    }
    if (bad && dev_status) atomicOr(dev_status, GRASS_DEV_BAD_INDEX);
    __syncthreads();  // bins zeroed by all threads before anyone adds (also closes the last stage)

    // stage 3: SJLT of the block; flat position q = a*kout + c (input-major flattening)
    float* orow = out + (int64_t)b * ld_out + L.out_offset;
    const float scale = 1.0f / sqrtf((float)s);
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float v = acc[i][j][e];
                const int a = tm * TM + wm * WM + i * 16 + (lane >> 2) + (e >> 1) * 8;
                const int c = tn * TN + wn * WN + j * 8 + (lane & 3) * 2 + (e & 1);
                if (a < kin && c < kout && v != 0.0f) {
                    const uint64_t q = (uint64_t)a * (uint64_t)kout + (uint64_t)c;
                    for (uint32_t r = 0; r < s; ++r) {
                        const uint64_t h = sjlt_hash_counter(seed, q * s + r + 1);
                        const uint32_t bk = sjlt_bucket(h, k);
                        const float sv = (s == 1) ? sjlt_signed(h, v) : sjlt_signed(h, v) * scale;
                        if (smem_bins) atomicAdd(&bins[bk], sv);
                        else atomicAdd(orow + bk, sv);
                    }
                }
            }
    if (smem_bins) {
        __syncthreads();
        for (uint32_t i = tid; i < k; i += kFgThreads) {
            const float v = bins[i];
            if (v != 0.0f) atomicAdd(orow + i, v);
        }
    }
}

// zeroes every layer's [out_offset, out_offset + k) range of every sample row
__global__ void factgrass_zero_kernel(const LayerDesc* __restrict__ descs, const __grid_constant__ LayerDesc single,
                                      float* __restrict__ out, int64_t ld_out)
{
    const LayerDesc& L = descs ? descs[blockIdx.z] : single;
    float* orow = out + (int64_t)blockIdx.y * ld_out + L.out_offset;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < L.k; i += gridDim.x * blockDim.x) orow[i] = 0.0f;
}

constexpr size_t kMaxSmemBins = 160 * 1024;

static grass_status fill_desc(LayerDesc& d, const factgrass_layer& l, int tile, int32_t T)
{
    if (l.spec.k == 0 || l.spec.s == 0) return GRASS_ERR_INVALID_ARG;
    if (l.d_in <= 0 || l.d_out <= 0 || l.kin < 0 || l.kout < 0 || l.kin > l.d_in || l.kout > l.d_out)
        return GRASS_ERR_INVALID_ARG;
    if (l.out_offset < 0) return GRASS_ERR_INVALID_ARG;
    if ((l.kin > 0 && l.kout > 0 && T > 0) && (!l.A || !l.G || !l.mask_in || !l.mask_out)) return GRASS_ERR_INVALID_ARG;
    d.A = (const uint16_t*)l.A;
    d.G = (const uint16_t*)l.G;
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
    d.pad_ = 0;
    return GRASS_OK;
}

static int fg_env_int(const char* name, int dflt)
{
    const char* v = std::getenv(name);
    return v ? std::atoi(v) : dflt;
}

static grass_status run_factgrass(const factgrass_layer* layers, int32_t L, grass_dtype dt, int32_t B, int32_t T,
                                  const int64_t* tok_begin, const int32_t* tok_count, float* out, int64_t ld_out,
                                  void* workspace, size_t workspace_bytes, uint32_t* dev_status, cudaStream_t st)
{
    if (L < 0 || B < 0 || T < 0 || (L > 0 && !layers)) return GRASS_ERR_INVALID_ARG;
    if (dt == GRASS_F32) return GRASS_ERR_UNSUPPORTED;
    if (dt != GRASS_BF16) return GRASS_ERR_INVALID_ARG;
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
    // 64 x 64 block tiles (3 CTAs per SM); larger blocks are covered by several tiles whose shared rows
    // come from L2.  The 128 x 128 variant (1 CTA per SM) is kept for comparison runs.
    const int tile = fg_env_int("FACTGRASS_TILE", 64) == 128 && max_kk > 64 ? 128 : 64;

    const bool grouped = workspace != nullptr;
    if (!grouped && L != 1) return GRASS_ERR_INVALID_ARG;
    LayerDesc single;
    std::memset(&single, 0, sizeof single);
    LayerDesc* dev_descs = nullptr;
    int max_tiles = 1;
    if (grouped) {
        if (workspace_bytes < (size_t)L * sizeof(LayerDesc) || ((uintptr_t)workspace & 15)) return GRASS_ERR_INVALID_ARG;
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
        if (rc == GRASS_OK)
            rc = cuda_ok(cudaMemcpyAsync(workspace, host, (size_t)L * sizeof(LayerDesc), cudaMemcpyHostToDevice, st));
        if (host != stack_buf) std::free(host);
        if (rc != GRASS_OK) return rc;
        dev_descs = (LayerDesc*)workspace;
    } else {
        grass_status rc = fill_desc(single, layers[0], tile, T);
        if (rc != GRASS_OK) return rc;
        max_tiles = single.tiles_m * single.tiles_n;
    }

    // zero the output ranges (the compress kernel accumulates partial projections into them)
    {
        dim3 zg((max_k + 1023) / 1024 > 0 ? (max_k + 1023) / 1024 : 1, (unsigned)B, (unsigned)L);
        if (zg.x > 64) zg.x = 64;
        factgrass_zero_kernel<<<zg, 256, 0, st>>>(dev_descs, single, out, ld_out);
        if (launch_status() != GRASS_OK) return GRASS_ERR_CUDA;
    }
    if (T == 0 || max_tiles == 0) return GRASS_OK;

    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return GRASS_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GRASS_ERR_CUDA;

    // token chunks.  Every chunk pays a fixed projection epilogue (tile*tile hashes and a k-bin flush),
    // so chunks are as long as the machine allows: when there are fewer work items than resident CTA
    // slots the token sum is split just enough to fill one wave; otherwise just enough for ~8 waves
    // so that the last, partial wave costs little.
    const int64_t base_items = (int64_t)L * B * max_tiles;
    const int64_t slots = (int64_t)sms * (tile == 64 ? 3 : 1);
    const int min_chunk = 64;
    int64_t want = base_items < slots ? slots / base_items : (8 * slots + base_items - 1) / base_items;
    int64_t max_chunks = (T + min_chunk - 1) / min_chunk;
    if (want > max_chunks) want = max_chunks;
    if (want < 1) want = 1;
    int chunk_len = (int)((T + want - 1) / want);
    chunk_len = (chunk_len + kTokTile - 1) / kTokTile * kTokTile;
    chunk_len = fg_env_int("FACTGRASS_CHUNK", chunk_len);
    if (chunk_len < kTokTile) chunk_len = kTokTile;
    chunk_len = (chunk_len + kTokTile - 1) / kTokTile * kTokTile;
    const int nchunks = (T + chunk_len - 1) / chunk_len;

    const size_t bins_bytes = (size_t)max_k_smem * sizeof(float);
    dim3 grid((unsigned)(nchunks * max_tiles), (unsigned)B, (unsigned)L);
    auto launch = [&](auto kern, size_t stage_bytes) -> grass_status {
        const size_t smem = 2 * stage_bytes + bins_bytes;
        if (smem > 48 * 1024) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
                return GRASS_ERR_CUDA;
        }
        kern<<<grid, kFgThreads, smem, st>>>(dev_descs, single, B, T, tok_begin, tok_count, max_tiles, chunk_len, out,
                                             ld_out, dev_status);
        return launch_status();
    };
    if (tile == 64) return launch(factgrass_kernel<64, 64>, (size_t)kTokTile * (2 * (64 * 2 + 16)));
    return launch(factgrass_kernel<128, 128>, (size_t)kTokTile * (2 * (128 * 2 + 16)));
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
