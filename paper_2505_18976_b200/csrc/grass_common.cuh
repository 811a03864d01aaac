// Shared device-side pieces of the sm_100a compression kernels: the seed-defined
// SJLT hash (bucket, sign) recomputed in registers, bf16 helpers, launch checks.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/grass.h"

namespace grass {

constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ULL;

__host__ __device__ __forceinline__ uint64_t mix64(uint64_t x)
{
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ULL;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBULL;
    x ^= x >> 31;
    return x;
}

// Hash of counter c = j*s + r + 1 under `seed` (Section 3.1: the random output
// coordinate and sign that input position j draws).
__host__ __device__ __forceinline__ uint64_t sjlt_hash_counter(uint64_t seed, uint64_t counter)
{
    return mix64(seed + kGolden * counter);
}

__host__ __device__ __forceinline__ uint32_t sjlt_bucket(uint64_t h, uint32_t k)
{
#ifdef __CUDA_ARCH__
    return __umulhi((uint32_t)(h >> 32), k);
#else
    return (uint32_t)(((h >> 32) * (uint64_t)k) >> 32);
#endif
}

// value with the hash's sign applied: flips the fp32 sign bit when H is odd.
__device__ __forceinline__ float sjlt_signed(uint64_t h, float v)
{
    return __uint_as_float(__float_as_uint(v) ^ ((uint32_t)h << 31));
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b)
{
    return __uint_as_float((uint32_t)b << 16);
}

// Gathered (scattered, read-once) loads of one element.  On B200 a plain load of an untouched 128-byte line makes
// DRAM deliver the whole line; the L2::64B prefetch-size hint limits the fetch to the 64-byte half that holds the
// element (nothing fetches less), which is what a sparse mask wants.  L1::no_allocate: the data are used once.
__device__ __forceinline__ uint32_t gather_u32(const uint32_t* p)
{
    uint32_t v;
    asm("ld.global.nc.L1::no_allocate.L2::64B.b32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ uint16_t gather_u16(const uint16_t* p)
{
    uint16_t v;
    asm("ld.global.nc.L1::no_allocate.L2::64B.b16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}

__device__ __forceinline__ float elem_value(float x) { return x; }
__device__ __forceinline__ float elem_value(__nv_bfloat16 x) { return __bfloat162float(x); }

// final store of a compressed value: fp32, or bf16 rounded to nearest even (a cache of compressed vectors kept
// at half the size; everything before the store is fp32)
__device__ __forceinline__ void store_out(float* out, int64_t off, float v, int out_bf16)
{
    if (out_bf16) reinterpret_cast<__nv_bfloat16*>(out)[off] = __float2bfloat16_rn(v);
    else out[off] = v;
}

template <typename T> struct elem;
template <> struct elem<float> {
    static __device__ __forceinline__ float load(const float* p)
    {
        return __uint_as_float(gather_u32(reinterpret_cast<const uint32_t*>(p)));
    }
};
template <> struct elem<__nv_bfloat16> {
    static __device__ __forceinline__ float load(const __nv_bfloat16* p)
    {
        return bf16_bits_to_float(gather_u16(reinterpret_cast<const uint16_t*>(p)));
    }
};

// grass_compress with row staging for dense masks (grass_compress_rows.cu): whether the operands allow it, and
// the launch
bool compress_rows_fits(const void* g, size_t elem_bytes, int64_t p, int64_t ld, const uint32_t* idx, int64_t kprime,
                        uint32_t k, int64_t n);
grass_status launch_compress_rows(const void* g, grass_dtype dt, int64_t n, int64_t p, int64_t ld, const uint32_t* idx,
                                  int64_t kprime, const grass_sjlt_spec& sp, float* out, int64_t ld_out,
                                  uint32_t* dev_status, cudaStream_t st, int out_bf16);

// launch-shape override set through grass_set_tuning, or `dflt` while the key is on automatic
int64_t tuning(grass_tuning_key key, int64_t dflt);

inline grass_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? GRASS_OK : GRASS_ERR_CUDA; }

inline grass_status launch_status()
{
    return cuda_ok(cudaGetLastError());
}

}  // namespace grass
