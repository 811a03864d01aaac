// grass_score: scores[i, m] = <train[i, :], test[m, :]> (attribute stage, Section 2.1).
// The default path is the tensor-core kernel (split-bf16 products in tensor memory, see
// grass_score_tc.cu); it loads with TMA and therefore wants 16-byte aligned bases and row strides.  This
// file holds the entry point and the plain fp32 FMA kernel (128 x 128 output tile per CTA, 8 x 8 per
// thread, 16-deep k tiles double-buffered through registers and shared memory) that takes every other
// input (and D = 0); the GRASS_TUNE_SCORE_FFMA override selects it for comparison runs.
#include "grass_common.cuh"

#include <cstdlib>
#include <cstring>

namespace grass {

constexpr int SC_BM = 128, SC_BN = 128, SC_BK = 16, SC_THREADS = 256, SC_PAD = 4;

// loads 4 consecutive floats of a row, zero beyond D / beyond the last row
__device__ __forceinline__ float4 load4_guarded(const float* __restrict__ base, int64_t row, int64_t rows,
                                                int64_t ld, int64_t d, int64_t D, bool vec_ok)
{
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row >= rows) return v;
    const float* p = base + row * ld + d;
    if (vec_ok && d + 3 < D) return __ldg(reinterpret_cast<const float4*>(p));
    if (d + 0 < D) v.x = __ldg(p + 0);
    if (d + 1 < D) v.y = __ldg(p + 1);
    if (d + 2 < D) v.z = __ldg(p + 2);
    if (d + 3 < D) v.w = __ldg(p + 3);
    return v;
}

__global__ void __launch_bounds__(SC_THREADS)
grass_score_kernel(const float* __restrict__ train, int64_t N, int64_t ld_train, const float* __restrict__ test,
                   int64_t M, int64_t ld_test, int64_t D, float* __restrict__ scores, int64_t ld_s, int vec_ok)
{
    __shared__ __align__(16) float As[2][SC_BK][SC_BM + SC_PAD];
    __shared__ __align__(16) float Bs[2][SC_BK][SC_BN + SC_PAD];

    const int tid = threadIdx.x;
    const int64_t n0 = (int64_t)blockIdx.x * SC_BM;
    const int64_t m0 = (int64_t)blockIdx.y * SC_BN;
    const int ty = tid / 16, tx = tid % 16;

    // each thread stages 2 float4 of each operand per k tile: rows lr and lr + 64, k quad lq
    const int lr = tid / 4, lq = tid % 4;
    float4 pa[2], pb[2];
    auto fetch = [&](int64_t d0) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            pa[h] = load4_guarded(train, n0 + lr + 64 * h, N, ld_train, d0 + lq * 4, D, vec_ok);
            pb[h] = load4_guarded(test, m0 + lr + 64 * h, M, ld_test, d0 + lq * 4, D, vec_ok);
        }
    };
    auto stash = [&](int buf) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int r = lr + 64 * h;
            As[buf][lq * 4 + 0][r] = pa[h].x; As[buf][lq * 4 + 1][r] = pa[h].y;
            As[buf][lq * 4 + 2][r] = pa[h].z; As[buf][lq * 4 + 3][r] = pa[h].w;
            Bs[buf][lq * 4 + 0][r] = pb[h].x; Bs[buf][lq * 4 + 1][r] = pb[h].y;
            Bs[buf][lq * 4 + 2][r] = pb[h].z; Bs[buf][lq * 4 + 3][r] = pb[h].w;
        }
    };

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    fetch(0);
    int buf = 0;
    for (int64_t d0 = 0; d0 < D; d0 += SC_BK, buf ^= 1) {
        stash(buf);
        __syncthreads();
        if (d0 + SC_BK < D) fetch(d0 + SC_BK);
#pragma unroll
        for (int kk = 0; kk < SC_BK; ++kk) {
            const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][kk][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[buf][kk][64 + tx * 4]);
            const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }

#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t row = n0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (row >= N) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int64_t col = m0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4));
            if (col < M) scores[row * ld_s + col] = acc[i][j];
        }
    }
}

grass_status launch_score_tc(const float* train, int64_t N, int64_t ld_train, const float* test, int64_t M,
                             int64_t ld_test, int64_t D, float* scores, int64_t ld_s, cudaStream_t st);
bool score_tc_supported(const float* train, int64_t ld_train, const float* test, int64_t ld_test, int64_t D);
grass_status launch_score_bf16(const void* train, int64_t N, int64_t ld_train, const void* test, int64_t M,
                               int64_t ld_test, int64_t D, float* scores, int64_t ld_s, cudaStream_t st);
bool score_bf16_supported(const void* train, int64_t ld_train, const void* test, int64_t ld_test, int64_t D);

// fp32 -> bf16, round to nearest even, row by row
__global__ void to_bf16_kernel(const float* __restrict__ in, int64_t n, int64_t k, int64_t ld_in,
                               __nv_bfloat16* __restrict__ out, int64_t ld_out)
{
    const int64_t i = blockIdx.y;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k; j += (int64_t)gridDim.x * blockDim.x)
        out[i * ld_out + j] = __float2bfloat16_rn(in[i * ld_in + j]);
}

}  // namespace grass

extern "C" grass_status grass_score(const float* train, int64_t N, int64_t ld_train, const float* test, int64_t M,
                                    int64_t ld_test, int64_t D, float* scores, int64_t ld_s, void* stream)
{
    if (N < 0 || M < 0 || D < 0 || ld_train < D || ld_test < D || ld_s < M) return GRASS_ERR_INVALID_ARG;
    if (N == 0 || M == 0) return GRASS_OK;
    if (!scores || (D > 0 && (!train || !test))) return GRASS_ERR_INVALID_ARG;
    if (grass::tuning(GRASS_TUNE_SCORE_FFMA, 0) == 0 && grass::score_tc_supported(train, ld_train, test, ld_test, D))
        return grass::launch_score_tc(train, N, ld_train, test, M, ld_test, D, scores, ld_s, (cudaStream_t)stream);
    const int64_t gx = (N + grass::SC_BM - 1) / grass::SC_BM, gy = (M + grass::SC_BN - 1) / grass::SC_BN;
    if (gx > 0x7FFFFFFFLL || gy > 65535) return GRASS_ERR_UNSUPPORTED;
    const int vec_ok = ((uintptr_t)train % 16 == 0) && ((uintptr_t)test % 16 == 0) && (ld_train % 4 == 0) &&
                       (ld_test % 4 == 0);
    dim3 grid((unsigned)gx, (unsigned)gy);
    grass::grass_score_kernel<<<grid, grass::SC_THREADS, 0, (cudaStream_t)stream>>>(
        train, N, ld_train, test, M, ld_test, D, scores, ld_s, vec_ok);
    return grass::launch_status();
}

extern "C" grass_status grass_to_bf16(const float* in, int64_t n, int64_t k, int64_t ld_in, void* out, int64_t ld_out,
                                      void* stream)
{
    if (n < 0 || k < 0 || ld_in < k || ld_out < k) return GRASS_ERR_INVALID_ARG;
    if (n == 0 || k == 0) return GRASS_OK;
    if (!in || !out) return GRASS_ERR_INVALID_ARG;
    if (n > 65535) return GRASS_ERR_UNSUPPORTED;
    int64_t gx = (k + 1023) / 1024;
    if (gx > 1024) gx = 1024;
    dim3 grid((unsigned)gx, (unsigned)n);
    grass::to_bf16_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(in, n, k, ld_in, (__nv_bfloat16*)out, ld_out);
    return grass::launch_status();
}

extern "C" grass_status grass_score_bf16(const void* train, int64_t N, int64_t ld_train, const void* test, int64_t M,
                                         int64_t ld_test, int64_t D, float* scores, int64_t ld_s, void* stream)
{
    if (N < 0 || M < 0 || D < 0 || ld_train < D || ld_test < D || ld_s < M) return GRASS_ERR_INVALID_ARG;
    if (N == 0 || M == 0) return GRASS_OK;
    if (!scores || (D > 0 && (!train || !test))) return GRASS_ERR_INVALID_ARG;
    if (D == 0)
        return grass::cuda_ok(cudaMemset2DAsync(scores, (size_t)ld_s * sizeof(float), 0, (size_t)M * sizeof(float),
                                                (size_t)N, (cudaStream_t)stream));
    if (!grass::score_bf16_supported(train, ld_train, test, ld_test, D)) return GRASS_ERR_UNSUPPORTED;
    return grass::launch_score_bf16(train, N, ld_train, test, M, ld_test, D, scores, ld_s, (cudaStream_t)stream);
}
