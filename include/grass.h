/*
 * grass.h -- C ABI of the B200 (sm_100a) gradient-compression library.
 *
 * The calls follow the problem statement of "GraSS: Scalable Data Attribution
 * with Gradient Sparsification and Sparse Projection" (arXiv 2505.18976):
 *
 *   grass_compress               SJLT_k o Mask_k'      on dense per-sample gradients (Section 3.3.1)
 *   factgrass_compress           SJLT_k o Mask_{k'_in (x) k'_out} for one linear layer (Section 3.3.2)
 *   factgrass_compress_grouped   the same for many layers in one launch
 *   grass_score                  all-pair inner products of compressed vectors (Section 2.1, attribute stage)
 *   grass_to_bf16, grass_score_bf16   the same for a cache stored in bf16
 *
 * Conventions (all calls):
 *   - Pointers are DEVICE pointers unless the parameter is marked "host".  The caller owns every
 *     buffer; the library allocates nothing and keeps no state between calls (the only exception is the
 *     table of launch-shape overrides behind grass_set_tuning, a test hook that is empty unless set).
 *     The library never reads the process environment.
 *   - The gathered inputs (g of grass_compress / grass_mask, A and G of the factgrass / factmask calls) may
 *     also be page-locked host memory that the device can address (cudaHostAlloc, cudaHostRegister): the
 *     kernels then read the masked elements in place across the bus, 64 bytes per touched piece, which for a
 *     sparse mask moves far less than copying the inputs would.  Every other buffer is device memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Work is
 *     enqueued on it and the call returns without synchronising, except where stated.
 *   - Output buffers are OVERWRITTEN (the call zeroes them itself where its kernels accumulate).
 *   - Arguments that can be checked on the host (null pointers, negative sizes, k == 0, s == 0,
 *     k' > p, strides shorter than the row) are rejected with GRASS_ERR_INVALID_ARG before any
 *     launch.  Launch failures return GRASS_ERR_CUDA.  Faults only visible on the device (a mask
 *     index >= p, a bounded wait that expired) never trap or hang: the offending element is skipped
 *     and a bit is OR-ed into *dev_status (nullable; the caller zeroes and reads it).
 *   - Zero-size calls (n == 0, B == 0, T == 0 ...) are valid and leave a zeroed / untouched output.
 *   - Mask index lists are uint32, strictly ascending, < p ("exactly one non-repetitive non-zero
 *     entry per row" of the selection matrix, Section 3.2).  They are shared by all samples of a call.
 *     A NULL mask is the identity and requires the masked length to equal the row length.
 *
 * The sparse projection (Section 3.1) is defined by a seed, not by stored indices.  For input
 * position j (position in the MASKED vector) and draw r < s:
 *       H      = mix64(seed + 0x9E3779B97F4A7C15 * (j*s + r + 1))        (SplitMix64 stream)
 *       bucket = ((H >> 32) * k) >> 32,   sign = (H & 1) ? -1 : +1
 *       out[bucket] += sign * value / sqrt(s)
 */
#ifndef GRASS_H_
#define GRASS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GRASS_OK = 0,
    GRASS_ERR_INVALID_ARG = 1,
    GRASS_ERR_BAD_MASK = 2,
    GRASS_ERR_UNSUPPORTED = 3,
    GRASS_ERR_CUDA = 4,
    GRASS_ERR_TIMEOUT = 5
} grass_status;

typedef enum { GRASS_F32 = 0, GRASS_BF16 = 1 } grass_dtype;

/* bits OR-ed into *dev_status by kernels */
#define GRASS_DEV_BAD_INDEX 1u   /* a mask index was >= the row length; that element was skipped */
#define GRASS_DEV_TIMEOUT   2u   /* a bounded on-device wait expired */
#define GRASS_DEV_BAD_LENGTH 4u  /* a per-sample token count was outside [0, T_max]; it was clamped */
#define GRASS_DEV_NOT_PD    8u   /* grass_fim_factor met a pivot <= 0: F + lambda I is not positive definite */

/* SJLT_k with s non-zeros per column of the projection matrix (Section 3.1).  k >= 1, s >= 1. */
typedef struct {
    uint32_t k;
    uint32_t s;
    uint64_t seed;
} grass_sjlt_spec;

/*
 * GraSS (Section 3.3.1): out[i, :] = SJLT_{k,s,seed}( g[i, idx[0..kprime)] ),  i in [0, n).
 *   g        n x p, row-major, row stride `ld` elements (ld >= p), dtype `dt` (fp32 or bf16).
 *   idx      kprime ascending coordinates (Random or Selective Mask, Section 3.2); NULL means the
 *            identity mask and requires kprime == p (plain SJLT, the k' = p case of Section 3.3.1).
 *   out      n x spec->k fp32, row stride ld_out >= k.  Overwritten.
 *   The masked vector is never written to memory: gather and scatter-add are one kernel.
 */
grass_status grass_compress(const void* g, grass_dtype dt, int64_t n, int64_t p, int64_t ld,
                            const uint32_t* idx, int64_t kprime, const grass_sjlt_spec* spec /*host*/,
                            float* out, int64_t ld_out, uint32_t* dev_status, void* stream);

/*
 * FactGraSS for one linear layer (Section 3.3.2, stages 1-3; Eq. 2 with selection matrices):
 *   out[b, :] = SJLT( vec( sum_t A[b,t,mask_in] (x) G[b,t,mask_out] ) ),  flat index a*kout + c.
 *   A   B x T x d_in   layer inputs,            token-major contiguous, dtype dt (bf16 or fp32)
 *   G   B x T x d_out  pre-activation gradients, token-major contiguous, same dtype
 *   out B x spec->k fp32, row stride ld_out.  Overwritten.
 * The kin x kout block is accumulated in fp32 on tensor cores (tensor memory) and never reaches
 * HBM.  fp32 factors are split exactly into three bf16 pieces each and contracted with six partial
 * products, which keeps fp32 accuracy.
 */
grass_status factgrass_compress(const void* A, const void* G, grass_dtype dt, int32_t B, int32_t T,
                                int32_t d_in, int32_t d_out, const uint32_t* mask_in, int32_t kin,
                                const uint32_t* mask_out, int32_t kout,
                                const grass_sjlt_spec* spec /*host*/, float* out, int64_t ld_out,
                                uint32_t* dev_status, void* stream);

/* One linear layer of a grouped call.  Layer l writes out[b, out_offset .. out_offset + spec.k). */
typedef struct {
    const void* A;
    const void* G;
    const uint32_t* mask_in;
    const uint32_t* mask_out;
    int32_t d_in, d_out;
    int32_t kin, kout;
    grass_sjlt_spec spec;
    int64_t out_offset;
} factgrass_layer;

/*
 * FactGraSS over L layers that share B, T, dtype and the output matrix (the layer-wise compression
 * of Section 3.3.2: one compressed block per layer, concatenated per sample).
 *   layers     host array of L descriptors (device pointers inside).  It is copied to `workspace`
 *              on `stream`; the host array may be reused as soon as the call returns.
 *   workspace  device scratch of at least factgrass_grouped_workspace_bytes(L) bytes, 256-byte
 *              aligned, owned by the caller, in use until the work enqueued by this call has finished.
 *   out        B x ld_out fp32; each layer's [out_offset, out_offset + k) range is overwritten,
 *              ranges of different layers must not overlap.
 * A layer whose kin or kout is 0 contributes a zeroed output range and is otherwise skipped.
 * With L > 1 the descriptor table is copied from host memory owned by the call, so grouped calls
 * (this one, the _varlen, factmask and _static variants) must not be recorded into a CUDA stream capture;
 * a single layer (L == 1) travels as a kernel argument and has no such copy.
 */
grass_status factgrass_compress_grouped(const factgrass_layer* layers /*host*/, int32_t L, grass_dtype dt,
                                        int32_t B, int32_t T, float* out, int64_t ld_out,
                                        void* workspace, size_t workspace_bytes,
                                        uint32_t* dev_status, void* stream);
size_t factgrass_grouped_workspace_bytes(int32_t L);

/*
 * The same two compressors writing the compressed rows in a chosen precision (the paper leaves the storage
 * precision of the cache open; a bf16 cache is half the bytes and feeds grass_score_bf16 directly).
 *   out_dt   GRASS_F32: identical to grass_compress / factgrass_compress_grouped.
 *            GRASS_BF16: out is n x k (B x ld_out) bf16, ld_out in elements.  Everything up to the final store is
 *            the fp32 arithmetic of the fp32 calls; each output is rounded to nearest even exactly once.  That
 *            needs a launch in which one thread block or one cluster owns a whole row, so there are no partial
 *            sums in global memory: grass_compress_out then needs k small enough for shared-memory bins (k <=
 *            51,200); factgrass_compress_grouped_out needs k'_in, k'_out <= 64 (or a launch small enough for the
 *            cluster kernel: k'_in, k'_out <= 128), T <= 8,192 and k <= 40,960.  Anything else returns
 *            GRASS_ERR_UNSUPPORTED with nothing enqueued (use the fp32 call and grass_to_bf16).
 *   factgrass_compress_grouped_out accepts workspace == NULL for a single layer (L == 1).
 */
grass_status grass_compress_out(const void* g, grass_dtype dt, int64_t n, int64_t p, int64_t ld,
                                const uint32_t* idx, int64_t kprime, const grass_sjlt_spec* spec /*host*/,
                                void* out, grass_dtype out_dt, int64_t ld_out, uint32_t* dev_status, void* stream);
grass_status factgrass_compress_grouped_out(const factgrass_layer* layers /*host*/, int32_t L, grass_dtype dt,
                                            int32_t B, int32_t T, void* out, grass_dtype out_dt, int64_t ld_out,
                                            void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                                            void* stream);

/*
 * Sparsification alone (Section 3.2: Random / Selective Mask used as the whole compressor, which the
 * paper evaluates next to GraSS and FactGraSS).
 *   grass_mask         out[i, j] = g[i, idx[j]],  out n x kprime fp32 (row stride ld_out >= kprime);
 *                      g and idx as in grass_compress (idx must not be NULL; n <= 65,535 per call).
 *   factmask_compress  out[b, a*kout + c] = sum_t A[b,t,mask_in[a]] * G[b,t,mask_out[c]]: the k'_in x k'_out
 *                      block of Eq. 2 with selection matrices, flattened input-major, without projection.
 *                      out is B x (kin*kout) fp32; arguments as in factgrass_compress.
 *   factmask_compress_grouped  the same for L layers; layer l writes out[b, out_offset .. + kin*kout);
 *                      the `spec` member of the descriptors is ignored.
 * An index >= the row length gives 0 in grass_mask (and is skipped in factmask) and sets GRASS_DEV_BAD_INDEX.
 */
grass_status grass_mask(const void* g, grass_dtype dt, int64_t n, int64_t p, int64_t ld, const uint32_t* idx,
                        int64_t kprime, float* out, int64_t ld_out, uint32_t* dev_status, void* stream);
grass_status factmask_compress(const void* A, const void* G, grass_dtype dt, int32_t B, int32_t T, int32_t d_in,
                               int32_t d_out, const uint32_t* mask_in, int32_t kin, const uint32_t* mask_out,
                               int32_t kout, float* out, int64_t ld_out, uint32_t* dev_status, void* stream);
grass_status factmask_compress_grouped(const factgrass_layer* layers /*host*/, int32_t L, grass_dtype dt, int32_t B,
                                       int32_t T, float* out, int64_t ld_out, void* workspace,
                                       size_t workspace_bytes, uint32_t* dev_status, void* stream);

/*
 * FactGraSS on batches whose samples have their own sequence lengths.  The sum over tokens in Eq. 2
 * (Section 3.3.2) runs over the tokens of one sample; padding tokens are not part of it, so they are
 * not read at all.  A and G of every layer are token-major matrices (rows x d_in, rows x d_out); the
 * tokens of sample b are the tok_count[b] consecutive rows starting at row tok_begin[b].
 *   tok_begin  device array of B row indices, or NULL for a padded batch (tok_begin[b] = b * T_max).
 *   tok_count  device array of B token counts in [0, T_max], or NULL (every sample has T_max tokens).
 *              A count outside [0, T_max] is clamped and GRASS_DEV_BAD_LENGTH is OR-ed into *dev_status.
 *   T_max      upper bound of the counts (sizes the launch); with both arrays NULL the calls equal
 *              factgrass_compress / factgrass_compress_grouped.
 * A packed batch (no padding rows at all) is tok_begin = exclusive prefix sum of tok_count.
 * Everything else as in factgrass_compress / factgrass_compress_grouped; a sample with no tokens gets
 * a zero row.
 */
grass_status factgrass_compress_varlen(const void* A, const void* G, grass_dtype dt, int32_t B, int32_t T_max,
                                       const int64_t* tok_begin, const int32_t* tok_count, int32_t d_in,
                                       int32_t d_out, const uint32_t* mask_in, int32_t kin,
                                       const uint32_t* mask_out, int32_t kout,
                                       const grass_sjlt_spec* spec /*host*/, float* out, int64_t ld_out,
                                       uint32_t* dev_status, void* stream);
grass_status factgrass_compress_grouped_varlen(const factgrass_layer* layers /*host*/, int32_t L, grass_dtype dt,
                                               int32_t B, int32_t T_max, const int64_t* tok_begin,
                                               const int32_t* tok_count, float* out, int64_t ld_out,
                                               void* workspace, size_t workspace_bytes,
                                               uint32_t* dev_status, void* stream);

/*
 * factgrass_compress_grouped for callers that cannot hand over a device workspace.
 * (An engineering variant: the paper has no counterpart to it.)
 *
 * Some callers are not in a position to allocate device memory at the moment they need to compress:
 * a hook that runs in the middle of a backward pass under a framework whose memory pool already owns
 * all of HBM, a serving or training loop that must not hit the implicit device synchronisation of
 * cudaMalloc/cudaFree, or a plug-in whose host owns the allocator.  For them the layer descriptor
 * table -- the only scratch the grouped kernels use -- is a fixed array inside the library image
 * (22,528 bytes, resident on every GPU that loads the library until the process exits).  This call
 * performs no cudaMalloc, cudaFree or other allocation, on the device or through any library.
 *
 *   Same arguments and results as factgrass_compress_grouped, minus workspace / workspace_bytes.
 *   L may be at most FACTGRASS_STATIC_MAX_LAYERS (256); more returns GRASS_ERR_UNSUPPORTED with
 *   nothing enqueued.  Split larger models over several calls (each on the same stream).
 *   The first call on a device looks up the table's device address (once per device, with that device
 *   current); make that first call outside any stream capture.
 *   All calls on a device share the one table, and it keeps the previous call's descriptors until they
 *   are overwritten: every call rewrites the L entries it uses before its kernels read them, nothing
 *   else needs clearing.  Two calls whose GPU work can overlap (different streams, or different host
 *   threads without ordering) race on the table; keep calls to this entry point on one stream, or
 *   order them with events.
 */
#define FACTGRASS_STATIC_MAX_LAYERS 256
grass_status factgrass_compress_grouped_static(const factgrass_layer* layers /*host*/, int32_t L, grass_dtype dt,
                                               int32_t B, int32_t T, float* out, int64_t ld_out,
                                               uint32_t* dev_status, void* stream);

/*
 * Attribute-stage scores (Section 2.1): scores[i*ld_s + m] = <train[i, :], test[m, :]>.
 *   train N x D, test M x D, fp32 row-major with strides ld_train, ld_test >= D.
 *   scores N x M fp32 (train-major), row stride ld_s >= M.  Overwritten (columns beyond M are left alone).
 *   fp32-accurate products and fp32 accumulation; contractions longer than 16,384 are summed in runs of
 *   8,192 so that the relative accuracy does not degrade with D.  Whenever the contraction is split (long D,
 *   or few output tiles) the partial sums meet in the output, which the call first zeroes on the stream.
 * These are raw inner products of compressed gradients; preconditioning is the caller's.
 * The call has no dev_status argument: should one of the kernel's bounded waits ever expire, the output tile
 * of that thread block is filled with NaN (so the failure cannot pass for a score), its tensor memory is
 * released and the kernel returns.  grass_score_bf16 follows the same convention.
 */
grass_status grass_score(const float* train, int64_t N, int64_t ld_train, const float* test, int64_t M,
                         int64_t ld_test, int64_t D, float* scores, int64_t ld_s, void* stream);

/*
 * The same scores for a cache kept in bf16 (half the bytes of the attribute stage's inputs; the paper does not
 * fix the storage precision, this is an option beside the fp32 path):
 *   grass_to_bf16     out[i*ld_out + j] = bf16(in[i*ld_in + j]), round to nearest even; n <= 65,535 rows per call.
 *   grass_score_bf16  scores[i*ld_s + m] = <train[i, :], test[m, :]> for bf16 train (N x D) and test (M x D);
 *                     products are exact in fp32, accumulation as in grass_score; scores fp32, overwritten.
 *                     Bases must be 16-byte aligned and ld_train, ld_test multiples of 8 (the rows are read by
 *                     TMA); anything else returns GRASS_ERR_UNSUPPORTED with nothing enqueued.
 */
grass_status grass_to_bf16(const float* in, int64_t n, int64_t k, int64_t ld_in, void* out /* bf16 */, int64_t ld_out,
                           void* stream);
grass_status grass_score_bf16(const void* train /* bf16 */, int64_t N, int64_t ld_train, const void* test /* bf16 */,
                              int64_t M, int64_t ld_test, int64_t D, float* scores, int64_t ld_s, void* stream);

/*
 * Projected Fisher information matrix (Section 2.1, cache stage step 2):
 *   F[a*ld_f + b] = (1/n) * sum_i X[i*ld + a] * X[i*ld + b],   a, b in [0, k).
 *   X  n x k compressed gradients, fp32, row stride ld >= k (n >= 1).  For the layer-wise block-diagonal
 *      approximation of Section 3.3.2 pass one layer's column range: X + layer_offset, k = k_l, same ld.
 *   F  k x k fp32, row stride ld_f >= k.  Overwritten (full symmetric matrix).
 * The contraction over the n samples runs on tensor cores with fp32 accuracy (exact bf16 splits).
 */
grass_status grass_fim(const float* X, int64_t n, int64_t k, int64_t ld, float* F, int64_t ld_f, void* stream);

/*
 * Damped inverse-FIM-vector products (Section 2.1, cache stage step 3: g~ = F^-1 g; the damping term
 * lambda is the hyper-parameter of the paper's appendix on experiment details).
 *   grass_fim_factor  replaces the lower triangle of F by the Cholesky factor L of F + lambda*I
 *                     (lambda >= 0; the strict upper triangle is scratch: the 64 x 64 diagonal blocks keep the
 *                     inverses of their factors there, the rest is left as it was).
 *                     If a pivot is not positive, GRASS_DEV_NOT_PD is OR-ed into *dev_status (nullable)
 *                     and the result is meaningless; nothing traps.
 *   grass_fim_apply   overwrites each of the M rows b_m of Bm (M x k fp32, row stride ld_b >= k) by
 *                     (F + lambda*I)^-1 b_m, using the factor produced by grass_fim_factor.
 * Preconditioned scores <g_test, F^-1 g_i> = <F^-1 g_test, g_i>: apply to the (few) test rows, then call
 * grass_score(train, solved_test).  fp32 throughout: the relative error grows with the condition
 * number of F + lambda*I.
 */
grass_status grass_fim_factor(float* F, int64_t k, int64_t ld_f, float lambda, uint32_t* dev_status, void* stream);
grass_status grass_fim_apply(const float* L, int64_t k, int64_t ld_f, float* Bm, int64_t M, int64_t ld_b,
                             void* stream);

/*
 * The (bucket, sign) table of SJLT_{k,s,seed} for input positions [0, kprime), produced by the same
 * device code the compress kernels use: bucket[j*s + r], sign[j*s + r] (+1 / -1).  Both are device
 * buffers of kprime*s entries.  For tests and for callers that want to store the projection.
 */
grass_status grass_sjlt_table(const grass_sjlt_spec* spec /*host*/, int64_t kprime, uint32_t* bucket,
                              int8_t* sign, void* stream);

/*
 * Checks a device index list: strictly ascending and every entry < p.  SYNCHRONISES `stream`.
 * Returns GRASS_OK or GRASS_ERR_BAD_MASK.
 */
grass_status grass_validate_mask(const uint32_t* idx, int64_t kprime, int64_t p, void* stream);

/*
 * Random Mask (Section 3.2): kprime distinct coordinates of [0, p), uniform over subsets, ascending,
 * written to the HOST array idx_host.  Deterministic in `seed`.  Runs on the CPU (set-up, not hot path).
 */
grass_status grass_random_mask_host(int64_t p, int64_t kprime, uint64_t seed, uint32_t* idx_host /*host*/);

const char* grass_status_string(grass_status st);

/*
 * Launch-shape overrides (a test and measurement hook; the paper has no counterpart).  Every call above chooses
 * its launch shape from the problem size.  The parity tests compare several shapes of the same kernel and the
 * benchmark sweeps them, so each choice can be forced here.  value < 0 (GRASS_TUNE_AUTO) restores the automatic
 * choice.  The table is process-wide and read at launch time; it is not meant to be changed while other threads
 * are inside library calls.  Unknown keys return GRASS_ERR_INVALID_ARG.
 */
typedef enum {
    GRASS_TUNE_COMPRESS_SAMPLES = 0,   /* grass_compress: samples per thread block (1, 2, 4, 8) */
    GRASS_TUNE_COMPRESS_JSPLIT = 1,    /* grass_compress: thread blocks that share one sample's masked positions */
    GRASS_TUNE_COMPRESS_CLUSTER = 2,   /* grass_compress: 0 = reduce position splits with global reductions */
    GRASS_TUNE_COMPRESS_DENSE = 3,     /* grass_compress: 0 = no vector-load path for identity masks */
    GRASS_TUNE_FACTGRASS_TILE = 4,     /* factgrass: block tile 64 or 128 */
    GRASS_TUNE_FACTGRASS_CHUNK = 5,    /* factgrass: tokens per thread block */
    GRASS_TUNE_FACTGRASS_CARVEOUT = 6, /* factgrass: shared-memory carve-out in percent */
    GRASS_TUNE_SCORE_FFMA = 7,         /* grass_score: 1 = plain FMA kernel instead of the tensor-core one */
    GRASS_TUNE_SCORE_SPLITS = 8,       /* grass_score, grass_score_bf16: splits of the contraction */
    GRASS_TUNE_SPLIT_PRODUCTS = 9,     /* fp32 contractions: partial products per fp32 product (3, 4 or 6) */
    GRASS_TUNE_FACTGRASS_PATH = 10,    /* factgrass: 0 = streaming kernel, 1 = cluster kernel (see factgrass.cu) */
    GRASS_TUNE_COMPRESS_ROWS = 11,     /* grass_compress: 0 = never stage row segments in shared memory, 1 = wherever the operands allow */
    GRASS_TUNE_COMPRESS_LOADS = 12,    /* grass_compress gather path: loads in flight per thread (4, 8, 16) */
    GRASS_TUNE_COMPRESS_THREADS = 13,  /* grass_compress gather path: threads per block (256, 512, 1024) */
    GRASS_TUNE_COMPRESS_IDX_SMEM = 14, /* grass_compress gather path: 0 = never copy the index list into shared memory */
    GRASS_TUNE_SCORE_BF16_SOLO = 15,   /* grass_score_bf16: 0 = always thread-block pairs, also for M <= 256 */
    GRASS_TUNE_COUNT = 16
} grass_tuning_key;
#define GRASS_TUNE_AUTO (-1)
grass_status grass_set_tuning(grass_tuning_key key, int64_t value);

#ifdef __cplusplus
}
#endif
#endif /* GRASS_H_ */
