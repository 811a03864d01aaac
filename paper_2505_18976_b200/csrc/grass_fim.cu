// Projected Fisher information matrix and damped inverse-FIM-vector products (Section 2.1, cache stage
// steps 2 and 3; applied per layer block under the block-diagonal approximation of Section 3.3.2).
//
//   grass_fim         F = (1/n) sum_i g_i g_i^T over compressed gradients: the tensor-core contraction of
//                     the FactGraSS kernel with both factors equal to the gradient matrix (factgrass.cu).
//   grass_fim_factor  F + lambda I = L L^T, blocked right-looking Cholesky in fp32, in place (lower part;
//                     the diagonal blocks' upper triangles receive the inverses of the diagonal factors).
//   grass_fim_apply   rows b_m <- (L L^T)^-1 b_m by blocked forward and back substitution.
//
// The factorisation and the substitutions are plain fp32 FMA kernels on 64-wide blocks: a diagonal-block
// kernel (one CTA), a row-wise triangular solve against a diagonal block, and a 64 x 64-tile
// C -= A B^T / C -= A B update.  They are O(k^3) once per layer, next to O(n k^2) for the matrix itself.
#include "grass_common.cuh"

namespace grass {

grass_status launch_fim(const float* X, int64_t n, int64_t k, int64_t ld, float scale, float* F, int64_t ld_f,
                        cudaStream_t st);

namespace fim {

constexpr int NB = 64;

__global__ void add_damping_kernel(float* __restrict__ F, int64_t k, int64_t ld, float lambda)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < k) F[i * ld + i] += lambda;
}

// Unblocked Cholesky of the jb x jb diagonal block at (j0, j0), one CTA, followed by the inverse of the
// triangular factor.  On return the block's lower triangle holds Ljj and its strict upper triangle holds the
// strict lower triangle of Ljj^-1, transposed (the diagonal of the inverse is 1 / diag(Ljj)): the upper
// triangle of F is not used by anything else, and with the inverse at hand every triangular solve against
// this block becomes a small matrix product.  A pivot that is not positive sets GRASS_DEV_NOT_PD and is
// replaced by 1 so that nothing divides by zero.
__global__ void __launch_bounds__(NB)
potrf_diag_kernel(float* __restrict__ F, int64_t ld, int64_t j0, int jb, uint32_t* dev_status)
{
    __shared__ float a[NB][NB + 1];                    // as the block is stored: the factor, and the transposed
                                                       // inverse above the diagonal
    __shared__ __align__(16) float lrel[NB][NB];       // lrel[c][m] = L[c+1+m][c], zero beyond the last row
    __shared__ __align__(16) float colc[2][NB];
    __shared__ float rdiag[NB];
    const int j = threadIdx.x;
    float* blk = F + j0 * ld + j0;
    float col[NB];                                     // col[i] = A[i][j]; the loads are all in flight together
#pragma unroll
    for (int i = 0; i < NB; ++i)
        col[i] = (i < jb && j <= i) ? blk[(int64_t)i * ld + j] : ((i == j && i >= jb) ? 1.0f : 0.0f);
    // Unscaled right-looking elimination: the owner of column c publishes it as it stands, every later column
    // subtracts A[i][c] A[j][c] / pivot.  Entries above a column's diagonal take part in the arithmetic but are
    // never read as results, so the update needs no row predicate; columns are scaled by 1/sqrt(pivot) at the end.
    bool not_pd = false;
    float pivot = 1.0f;
#pragma unroll 1
    for (int c = 0; c < NB; ++c) {
        float* cc = colc[c & 1];
        if (j == c) {
#pragma unroll
            for (int i4 = 0; i4 < NB; i4 += 4)
                *reinterpret_cast<float4*>(&cc[i4]) = make_float4(col[i4], col[i4 + 1], col[i4 + 2], col[i4 + 3]);
        }
        __syncthreads();                               // colc is double-buffered: one barrier per column
        float d = cc[c];
        if (!(d > 0.0f)) { not_pd = true; d = 1.0f; }
        if (j == c) pivot = d;
        if (j > c) {
            const float w = -cc[j] * __frcp_rn(d);
#pragma unroll
            for (int i4 = 0; i4 < NB; i4 += 4) {
                const float4 l4 = *reinterpret_cast<const float4*>(&cc[i4]);
                col[i4 + 0] = fmaf(l4.x, w, col[i4 + 0]);
                col[i4 + 1] = fmaf(l4.y, w, col[i4 + 1]);
                col[i4 + 2] = fmaf(l4.z, w, col[i4 + 2]);
                col[i4 + 3] = fmaf(l4.w, w, col[i4 + 3]);
            }
        }
    }
    if (not_pd && j == 0 && dev_status) atomicOr(dev_status, GRASS_DEV_NOT_PD);
    {
        const float sd = sqrtf(pivot), rs = 1.0f / sd;
        rdiag[j] = rs;
#pragma unroll
        for (int i = 0; i < NB; ++i) if (i >= j) a[i][j] = (i > j) ? col[i] * rs : sd;
    }
    __syncthreads();
#pragma unroll 4
    for (int m = 0; m < NB; ++m) lrel[j][m] = (j + 1 + m < NB) ? a[j + 1 + m][j] : 0.0f;
    __syncthreads();
    // Inverse of the factor, thread j on column j, by column-oriented forward substitution.  t[m] holds the
    // running right-hand side of row c+1+m: the window slides down one row per step inside the FMAs, so every
    // register index is a compile-time constant while c stays a run-time loop.
    float t[NB];
#pragma unroll
    for (int i = 0; i < NB; ++i) t[i] = (i == j) ? 1.0f : 0.0f;
#pragma unroll 1
    for (int c = 0; c < NB; ++c) {
        const float x = t[0] * rdiag[c];
        if (c > j) a[j][c] = x;
        const float nx = -x;
#pragma unroll
        for (int m4 = 0; m4 < NB; m4 += 4) {
            const float4 l4 = *reinterpret_cast<const float4*>(&lrel[c][m4]);
            t[m4 + 0] = fmaf(l4.x, nx, t[m4 + 1]);
            t[m4 + 1] = fmaf(l4.y, nx, t[m4 + 2]);
            t[m4 + 2] = fmaf(l4.z, nx, t[m4 + 3]);
            t[m4 + 3] = (m4 + 4 < NB) ? fmaf(l4.w, nx, t[(m4 + 4) & (NB - 1)]) : 0.0f;
        }
    }
    __syncthreads();
#pragma unroll 8
    for (int r = 0; r < NB; ++r)
        if (r < jb && j < jb) blk[(int64_t)r * ld + j] = a[r][j];
}

// Rows of C (rows x jb, at the block's column offset) solved against the diagonal block through its stored
// inverse (see potrf_diag_kernel):  forward  x Ljj^T = c  ->  x = c (Ljj^-1)^T,   backward  x Ljj = c  ->
// x = c Ljj^-1.  64 rows per CTA, a 4 x 4 register tile of the product per thread.
template <bool BACKWARD>
__global__ void __launch_bounds__(256)
trsm_rows_kernel(const float* __restrict__ Ljj, int64_t ld_l, int jb, float* __restrict__ C, int64_t ld_c, int64_t rows)
{
    __shared__ __align__(16) float w[NB][NB + 4];    // w[p][q]: x[q] = sum_p c[p] * w[p][q]
    __shared__ __align__(16) float ct[NB][NB + 4];   // ct[p][r] = c[r][p]
    const int tid = threadIdx.x;
    const int64_t r0 = (int64_t)blockIdx.x * NB;
    float lraw[NB * NB / 256], craw[NB * NB / 256];
#pragma unroll
    for (int u = 0; u < NB * NB / 256; ++u) {        // all global loads first: they are independent
        const int e = tid + u * 256, i = e / NB, j = e % NB;
        lraw[u] = (i < jb && j < jb) ? Ljj[(int64_t)i * ld_l + j] : 0.0f;
        craw[u] = (j < jb && r0 + i < rows) ? C[(r0 + i) * ld_c + j] : 0.0f;
    }
#pragma unroll
    for (int u = 0; u < NB * NB / 256; ++u) {
        const int e = tid + u * 256, i = e / NB, j = e % NB;   // consecutive threads: consecutive columns
        float v = 0.0f;
        if (i < jb && j < jb) v = (i == j) ? 1.0f / lraw[u] : lraw[u];   // j > i: inverse entry (j, i); j < i: unused
        // inverse entry (row a, col b), a >= b, is stored at block position [b][a]
        if (!BACKWARD) { w[i][j] = (j >= i) ? v : 0.0f; }                        // w[p][q] = inv[q][p], p <= q
        else           { if (j >= i) w[j][i] = v; if (j > i) w[i][j] = 0.0f; }   // w[p][q] = inv[p][q], p >= q
        ct[j][i] = craw[u];
    }
    __syncthreads();
    const int ty = tid / 16, tx = tid % 16;          // rows ty*4.., outputs tx*4..
    float acc[4][4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = 0.0f;
#pragma unroll 8
    for (int p = 0; p < NB; ++p) {
        const float4 c4 = *reinterpret_cast<const float4*>(&ct[p][ty * 4]);
        const float4 w4 = *reinterpret_cast<const float4*>(&w[p][tx * 4]);
        const float c[4] = {c4.x, c4.y, c4.z, c4.w}, ww[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(c[u], ww[v], acc[u][v]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int64_t r = r0 + ty * 4 + u;
        if (r >= rows) continue;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int q = tx * 4 + v;
            if (q < jb) C[r * ld_c + q] = acc[u][v];
        }
    }
}

// C[i][j] -= sum_{q<K} A[i][q] * B(j, q), 64 x 64 tile per CTA, 4 x 4 per thread, K <= 64.
//   B_TRANS = false: B(j, q) = Bm[j * ldb + q]  (C -= A B^T);  true: B(j, q) = Bm[q * ldb + j]  (C -= A B).
//   LOWER: C is square, only tiles on or below the diagonal run and only entries j <= i are written.
template <bool B_TRANS, bool LOWER>
__global__ void __launch_bounds__(256)
gemm_sub_kernel(float* __restrict__ C, int64_t ldc, int64_t rows, int64_t cols, const float* __restrict__ A, int64_t lda,
                const float* __restrict__ Bm, int64_t ldb, int K)
{
    if (LOWER && blockIdx.x > blockIdx.y) return;
    __shared__ __align__(16) float as[NB][NB + 4];   // as[q][i]
    __shared__ __align__(16) float bs[NB][NB + 4];   // bs[q][j]
    const int tid = threadIdx.x;
    const int64_t i0 = (int64_t)blockIdx.y * NB, j0 = (int64_t)blockIdx.x * NB;
    {
        float av[NB * NB / 256], bv[NB * NB / 256];
#pragma unroll
        for (int u = 0; u < NB * NB / 256; ++u) {     // all global loads first: they are independent
            const int e = tid + u * 256, hi = e / NB, lo = e % NB;   // consecutive threads: consecutive addresses
            av[u] = (i0 + hi < rows && lo < K) ? A[(i0 + hi) * lda + lo] : 0.0f;
            if (!B_TRANS) bv[u] = (j0 + hi < cols && lo < K) ? Bm[(j0 + hi) * ldb + lo] : 0.0f;
            else bv[u] = (j0 + lo < cols && hi < K) ? Bm[(int64_t)hi * ldb + j0 + lo] : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < NB * NB / 256; ++u) {
            const int e = tid + u * 256, hi = e / NB, lo = e % NB;
            as[lo][hi] = av[u];
            if (!B_TRANS) bs[lo][hi] = bv[u]; else bs[hi][lo] = bv[u];
        }
    }
    __syncthreads();
    const int ty = tid / 16, tx = tid % 16;
    float acc[4][4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = 0.0f;
    for (int q = 0; q < K; ++q) {
        const float4 a4 = *reinterpret_cast<const float4*>(&as[q][ty * 4]);
        const float4 b4 = *reinterpret_cast<const float4*>(&bs[q][tx * 4]);
        const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int64_t i = i0 + ty * 4 + u;
        if (i >= rows) continue;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int64_t j = j0 + tx * 4 + v;
            if (j < cols && (!LOWER || j <= i)) C[i * ldc + j] -= acc[u][v];
        }
    }
}

static inline unsigned blocks(int64_t n) { return (unsigned)((n + NB - 1) / NB); }

}  // namespace fim
}  // namespace grass

extern "C" grass_status grass_fim(const float* X, int64_t n, int64_t k, int64_t ld, float* F, int64_t ld_f,
                                  void* stream)
{
    if (n <= 0 || k < 0 || ld < k || ld_f < k) return GRASS_ERR_INVALID_ARG;
    if (k == 0) return GRASS_OK;
    if (!X || !F) return GRASS_ERR_INVALID_ARG;
    if (n > 0x7FFFFFFFLL || ld > 0x7FFFFFFFLL) return GRASS_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemset2DAsync(F, (size_t)ld_f * sizeof(float), 0, (size_t)k * sizeof(float), (size_t)k, st) != cudaSuccess)
        return GRASS_ERR_CUDA;
    return grass::launch_fim(X, n, k, ld, 1.0f / (float)n, F, ld_f, st);
}

extern "C" grass_status grass_fim_factor(float* F, int64_t k, int64_t ld_f, float lambda, uint32_t* dev_status,
                                         void* stream)
{
    using namespace grass::fim;
    if (k < 0 || ld_f < k || !(lambda >= 0.0f)) return GRASS_ERR_INVALID_ARG;
    if (k == 0) return GRASS_OK;
    if (!F) return GRASS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (lambda != 0.0f) add_damping_kernel<<<(unsigned)((k + 255) / 256), 256, 0, st>>>(F, k, ld_f, lambda);
    for (int64_t j0 = 0; j0 < k; j0 += NB) {
        const int jb = (int)((k - j0) < NB ? (k - j0) : NB);
        potrf_diag_kernel<<<1, NB, 0, st>>>(F, ld_f, j0, jb, dev_status);
        const int64_t rest = k - j0 - jb;
        if (rest > 0) {
            float* panel = F + (j0 + jb) * ld_f + j0;            // rows below the diagonal block, its columns
            trsm_rows_kernel<false><<<blocks(rest), 256, 0, st>>>(F + j0 * ld_f + j0, ld_f, jb, panel, ld_f, rest);
            float* trail = F + (j0 + jb) * ld_f + (j0 + jb);
            dim3 g(blocks(rest), blocks(rest));
            gemm_sub_kernel<false, true><<<g, 256, 0, st>>>(trail, ld_f, rest, rest, panel, ld_f, panel, ld_f, jb);
        }
    }
    return grass::launch_status();
}

extern "C" grass_status grass_fim_apply(const float* Lf, int64_t k, int64_t ld_f, float* Bm, int64_t M, int64_t ld_b,
                                        void* stream)
{
    using namespace grass::fim;
    if (k < 0 || M < 0 || ld_f < k || ld_b < k) return GRASS_ERR_INVALID_ARG;
    if (k == 0 || M == 0) return GRASS_OK;
    if (!Lf || !Bm) return GRASS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    // L y = b, block column by block column: solve the diagonal block, then remove its contribution from
    // the columns to the right
    for (int64_t j0 = 0; j0 < k; j0 += NB) {
        const int jb = (int)((k - j0) < NB ? (k - j0) : NB);
        trsm_rows_kernel<false><<<blocks(M), 256, 0, st>>>(Lf + j0 * ld_f + j0, ld_f, jb, Bm + j0, ld_b, M);
        const int64_t rest = k - j0 - jb;
        if (rest > 0) {
            dim3 g(blocks(rest), blocks(M));
            gemm_sub_kernel<false, false><<<g, 256, 0, st>>>(Bm + j0 + jb, ld_b, M, rest, Bm + j0, ld_b,
                                                              Lf + (j0 + jb) * ld_f + j0, ld_f, jb);
        }
    }
    // L^T x = y, from the last block column to the first
    for (int64_t j0 = ((k - 1) / NB) * NB; j0 >= 0; j0 -= NB) {
        const int jb = (int)((k - j0) < NB ? (k - j0) : NB);
        trsm_rows_kernel<true><<<blocks(M), 256, 0, st>>>(Lf + j0 * ld_f + j0, ld_f, jb, Bm + j0, ld_b, M);
        if (j0 > 0) {
            dim3 g(blocks(j0), blocks(M));
            gemm_sub_kernel<true, false><<<g, 256, 0, st>>>(Bm, ld_b, M, j0, Bm + j0, ld_b, Lf + j0 * ld_f, ld_f, jb);
        }
    }
    return grass::launch_status();
}
