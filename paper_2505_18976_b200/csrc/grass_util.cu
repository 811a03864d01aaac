// Set-up and test surface: the device hash table dump, mask validation, the host-side
// Random Mask sampler (Section 3.2) and status strings.
#include "grass_common.cuh"

#include <algorithm>
#include <atomic>
#include <unordered_set>
#include <vector>

namespace grass {

// launch-shape overrides (grass_set_tuning); a negative entry means "automatic"
static std::atomic<int64_t> g_tuning[GRASS_TUNE_COUNT];
static std::atomic<bool> g_tuning_used{false};

int64_t tuning(grass_tuning_key key, int64_t dflt)
{
    if (!g_tuning_used.load(std::memory_order_acquire)) return dflt;
    const int64_t v = g_tuning[key].load(std::memory_order_relaxed);
    return v < 0 ? dflt : v;
}

__global__ void sjlt_table_kernel(uint32_t k, uint32_t s, uint64_t seed, int64_t total, uint32_t* __restrict__ bucket,
                                  int8_t* __restrict__ sign)
{
    // entry e = j*s + r uses counter e + 1
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        const uint64_t h = sjlt_hash_counter(seed, (uint64_t)e + 1);
        bucket[e] = sjlt_bucket(h, k);
        sign[e] = (h & 1) ? -1 : 1;
    }
}

__global__ void validate_mask_kernel(const uint32_t* __restrict__ idx, int64_t kprime, int64_t p, uint32_t* flag)
{
    bool bad = false;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < kprime;
         j += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t v = idx[j];
        if ((int64_t)v >= p) bad = true;
        if (j > 0 && idx[j - 1] >= v) bad = true;
    }
    if (bad) atomicOr(flag, 1u);
}

// a 4-byte flag for grass_validate_mask lives in mapped pinned host memory so the call needs no
// device allocation; it is created per call and released before returning
struct PinnedFlag {
    uint32_t* host = nullptr;
    uint32_t* dev = nullptr;
    bool ok = false;
    PinnedFlag()
    {
        if (cudaHostAlloc((void**)&host, sizeof(uint32_t), cudaHostAllocMapped) != cudaSuccess) return;
        *host = 0;
        ok = cudaHostGetDevicePointer((void**)&dev, host, 0) == cudaSuccess;
    }
    ~PinnedFlag()
    {
        if (host) cudaFreeHost(host);
    }
};

}  // namespace grass

extern "C" grass_status grass_sjlt_table(const grass_sjlt_spec* spec, int64_t kprime, uint32_t* bucket, int8_t* sign,
                                         void* stream)
{
    if (!spec || spec->k == 0 || spec->s == 0 || kprime < 0) return GRASS_ERR_INVALID_ARG;
    if (kprime == 0) return GRASS_OK;
    if (!bucket || !sign) return GRASS_ERR_INVALID_ARG;
    const int64_t total = kprime * (int64_t)spec->s;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    grass::sjlt_table_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(spec->k, spec->s, spec->seed, total,
                                                                                 bucket, sign);
    return grass::launch_status();
}

extern "C" grass_status grass_validate_mask(const uint32_t* idx, int64_t kprime, int64_t p, void* stream)
{
    if (kprime < 0 || p < 0) return GRASS_ERR_INVALID_ARG;
    if (kprime > p) return GRASS_ERR_BAD_MASK;
    if (kprime == 0) return GRASS_OK;
    if (!idx) return GRASS_ERR_INVALID_ARG;
    grass::PinnedFlag flag;
    if (!flag.ok) return GRASS_ERR_CUDA;
    int64_t blocks = (kprime + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    grass::validate_mask_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(idx, kprime, p, flag.dev);
    if (grass::launch_status() != GRASS_OK) return GRASS_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return GRASS_ERR_CUDA;
    return *flag.host ? GRASS_ERR_BAD_MASK : GRASS_OK;
}

extern "C" grass_status grass_random_mask_host(int64_t p, int64_t kprime, uint64_t seed, uint32_t* idx_host)
{
    if (p < 0 || kprime < 0 || kprime > p || p >= 0xFFFFFFFFLL) return GRASS_ERR_INVALID_ARG;
    if (kprime == 0) return GRASS_OK;
    if (!idx_host) return GRASS_ERR_INVALID_ARG;
    // Subset sampling after R. Floyd: walk i over the last kprime values of [0, p); draw t uniformly
    // from [0, i]; keep t unless it is already chosen, in which case keep i.  Every kprime-subset is
    // equally likely.  The draws come from the same SplitMix64 mixing as the projection hash.
    std::unordered_set<uint32_t> chosen;
    chosen.reserve((size_t)kprime * 2);
    std::vector<uint32_t> picks;
    picks.reserve((size_t)kprime);
    const uint64_t stream_seed = seed ^ 0xD1B54A32D192ED03ULL;
    for (int64_t i = p - kprime; i < p; ++i) {
        const uint64_t x = grass::mix64(stream_seed + grass::kGolden * ((uint64_t)i + 1));
        const uint32_t t = (uint32_t)(((unsigned __int128)x * (unsigned __int128)((uint64_t)i + 1)) >> 64);
        const uint32_t pick = chosen.count(t) ? (uint32_t)i : t;
        chosen.insert(pick);
        picks.push_back(pick);
    }
    std::sort(picks.begin(), picks.end());
    std::copy(picks.begin(), picks.end(), idx_host);
    return GRASS_OK;
}

extern "C" grass_status grass_set_tuning(grass_tuning_key key, int64_t value)
{
    if ((int)key < 0 || (int)key >= (int)GRASS_TUNE_COUNT) return GRASS_ERR_INVALID_ARG;
    if (!grass::g_tuning_used.load(std::memory_order_acquire)) {
        // first use: every key starts on automatic
        for (int i = 0; i < (int)GRASS_TUNE_COUNT; ++i) grass::g_tuning[i].store(-1, std::memory_order_relaxed);
        grass::g_tuning_used.store(true, std::memory_order_release);
    }
    grass::g_tuning[key].store(value < 0 ? -1 : value, std::memory_order_relaxed);
    return GRASS_OK;
}

extern "C" const char* grass_status_string(grass_status st)
{
    switch (st) {
        case GRASS_OK: return "ok";
        case GRASS_ERR_INVALID_ARG: return "invalid argument";
        case GRASS_ERR_BAD_MASK: return "mask indices not strictly ascending or out of range";
        case GRASS_ERR_UNSUPPORTED: return "unsupported dtype or size";
        case GRASS_ERR_CUDA: return "CUDA error";
        case GRASS_ERR_TIMEOUT: return "bounded device wait expired";
        default: return "unknown status";
    }
}
