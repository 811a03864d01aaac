// Pieces shared by the FactGraSS kernels (factgrass.cu: the streaming kernel; factgrass_cluster.cu: the
// cluster kernel for launches of about one wave): the per-layer descriptor and the register -> operand-tile
// packing.
#pragma once

#include "grass_common.cuh"
#include "tcgen05_util.cuh"

namespace grass {

constexpr int kFgThreads = 256;
constexpr int kTokTile = 32;  // tokens per pipeline stage
constexpr int kFgBufs = 2;    // operand-tile buffers per CTA

struct LayerDesc {
    const void* A;
    const void* G;
    const uint32_t* mask_in;
    const uint32_t* mask_out;
    int32_t d_in, d_out;
    int32_t kin, kout;
    uint32_t k, s;
    uint64_t seed;
    int64_t out_offset;
    int32_t tiles_m, tiles_n;
    int32_t use_smem_bins;
    float scale;   // raw-block epilogue: factor applied to every entry
};
static_assert(sizeof(LayerDesc) == 88, "descriptor layout");

// Token tile staged per pipeline step = the k extent of one shared-memory operand tile.
static_assert(kTokTile == tc::BK, "a stage holds one operand tile of 32 tokens");

template <bool F32> struct in_elem { using type = uint16_t; };
template <> struct in_elem<true> { using type = uint32_t; };

// eight consecutive tokens of one masked column (bf16 bit patterns, one per register) -> the 16-byte
// K-major chunk of that operand row
__device__ __forceinline__ uint4 pack8_bf16(const uint32_t (&v)[8])
{
    return make_uint4(v[0] | (v[1] << 16), v[2] | (v[3] << 16), v[4] | (v[5] << 16), v[6] | (v[7] << 16));
}

constexpr size_t kMaxSmemBins = 160 * 1024;   // k-bin accumulators up to this size live in shared memory

// The cluster kernel: one thread-block cluster per (layer, sample); see factgrass_cluster.cu.
// cluster_path_fits says whether every layer of the call can take it (one block tile per sample, bins in shared
// memory) and how many resident thread blocks per SM it would have.
struct ClusterPlan {
    int tile_m, tile_n;   // block tile (64 or 128 each)
    int per_sm;           // resident thread blocks per SM
    size_t smem;          // dynamic shared memory per thread block
};
bool cluster_path_fits(const LayerDesc* host_descs, int32_t L, ClusterPlan* plan);
grass_status launch_factgrass_cluster(const LayerDesc* dev_descs, const LayerDesc& single, const ClusterPlan& plan,
                                      int32_t L, int32_t B, int32_t T, const int64_t* tok_begin,
                                      const int32_t* tok_count, int32_t nc, int32_t chunk_len, float* out,
                                      int64_t ld_out, uint32_t* dev_status, cudaStream_t st, int out_bf16);

}  // namespace grass
