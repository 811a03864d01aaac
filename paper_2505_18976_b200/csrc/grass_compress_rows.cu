// grass_compress for dense masks (Section 3.3.1 with a mask that touches most of every row): row staging.
//
// When a mask keeps one coordinate in sixteen or more, almost every 64-byte piece of a row holds a masked
// element, so gathering element by element moves the whole row anyway -- one dependent 4-byte load per element,
// issued only after the mask indices have arrived, by thread blocks that all run the same phases at once.
// Here one thread block owns one sample and walks its row in windows of 16 KB: one thread keeps four windows
// of bulk copies (cp.async.bulk, completion on an mbarrier) in flight, starting the moment the block starts, with
// no dependency on the mask.  The index list itself is brought into shared memory by one more bulk copy (every
// thread block reads all of it: from global memory that is hundreds of thread blocks asking L2 for the same lines);
// the warps then find the mask positions at which the windows begin (32-way search in the ascending list).  When
// a window has landed, the threads pick its masked elements from shared memory; each warp compacts the non-zero
// ones into a small queue, so that every lane hashes a non-zero (Section 3.1: the cost of the projection follows
// the non-zeros), and adds them into the k-bin accumulator while the next windows are still streaming in.
// A row is finished by the thread block that started it: no cluster, no zero-fill, no global atomics, one store of
// the bins.
// Measured on B200 (256 x 65,536 fp32, mask 1/8): 28.6 us per call against 26.5 us for the gather kernel.  The copies
// alone stream the 67 MB in about 13 us: a staging kernel can only keep as many bytes in flight as shared memory
// holds (64 KB per thread block here, about 16-19 MB over the GPU), which is just the latency-bandwidth product
// of HBM under load, and every window's processing delays its buffer's refill.  The gather kernel has all loads of
// the launch in flight at once.  The path is therefore kept as an option (GRASS_TUNE_COMPRESS_ROWS = 1), not
// as the default.
// Needs 16-byte aligned rows and index list, at most 32 windows per row (p <= 131,072 fp32 / 262,144 bf16
// coordinates), an index list of at most 48 KB and enough samples to fill the machine; everything else takes the
// gather kernel in grass_compress.cu.
#include "grass_common.cuh"
#include "tcgen05_util.cuh"

namespace grass {

constexpr int kRowsThreads = 256;
constexpr int kRowsWarps = kRowsThreads / 32;
constexpr int kWinBytes = 16 * 1024;           // window of a row staged at a time
constexpr int kWinBufs = 4;                    // windows in flight
constexpr int kMaxWins = 32;                   // windows per row
constexpr int kMaxIdxBytes = 48 * 1024;        // index list kept in shared memory
constexpr int kRowsU = 2;                      // positions per thread and round
constexpr int kQueue = 32 * kRowsU;            // per-warp queue of non-zero entries: one round always fits

// smallest j in [0, n) with idx[j] >= target (n if there is none), by a whole warp: 32 probes per round.
// idx is the copy of the index list in shared memory.
__device__ __forceinline__ int64_t warp_lower_bound(const uint32_t* idx, int64_t n, uint64_t target)
{
    const int lane = threadIdx.x & 31;
    int64_t lo = 0, hi = n;                     // the answer lies in [lo, hi]
    while (hi - lo > 32) {
        const int64_t step = (hi - lo + 31) / 32;
        const int64_t q = lo + (int64_t)lane * step;
        const bool below = q < hi && (uint64_t)idx[q] < target;
        const int cnt = __popc(__ballot_sync(0xFFFFFFFFu, below));      // probes are ascending: a prefix is below
        if (cnt == 0) { hi = lo; break; }
        const int64_t last_below = lo + (int64_t)(cnt - 1) * step;
        const int64_t first_not = lo + (int64_t)cnt * step;
        lo = last_below + 1;
        hi = first_not < hi ? first_not : hi;
    }
    const int64_t q = lo + lane;
    const bool below = q < hi && (uint64_t)idx[q] < target;
    return lo + __popc(__ballot_sync(0xFFFFFFFFu, below));
}

using tc::bulk_copy;
using tc::expect_tx;

template <typename T, bool S1>
__global__ void __launch_bounds__(kRowsThreads)
grass_compress_rows_kernel(const T* __restrict__ g, int64_t p, int64_t ld, const uint32_t* __restrict__ idx,
                           int64_t kprime, uint32_t k, uint32_t s, uint64_t seed, float scale,
                           float* __restrict__ out, int64_t ld_out, uint32_t idx_smem_bytes, uint32_t* dev_status,
                           int out_bf16)
{
    constexpr int64_t WIN = kWinBytes / (int)sizeof(T);      // coordinates per window
    // [kWinBufs windows][index list][k bins][per-warp queues: value, position]
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[kWinBufs + 1];
    __shared__ int64_t jb[kMaxWins + 1];                     // window w holds mask positions [jb[w], jb[w + 1])
    uint32_t* sidx = reinterpret_cast<uint32_t*>(smem + kWinBufs * kWinBytes);
    float* bins = reinterpret_cast<float*>(smem + kWinBufs * kWinBytes + idx_smem_bytes);
    float* qval = bins + (k + 3) / 4 * 4;
    uint32_t* qpos = reinterpret_cast<uint32_t*>(qval + kRowsWarps * kQueue);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t i = blockIdx.x;
    const T* row = g + i * ld;
    const int nwin = (int)((p + WIN - 1) / WIN);             // <= kMaxWins (checked by the launcher)
    const uint32_t bar0 = tc::smem_u32(&bars[0]), bar_idx = bar0 + 8 * kWinBufs;
    const uint32_t buf0 = tc::smem_u32(smem);
    const uint32_t idx_bulk = (uint32_t)((kprime * 4) & ~(int64_t)15);   // the part whole 16-byte copies cover

    // bytes of window w that whole 16-byte copies cover; the few elements behind them are loaded directly
    auto bulk_bytes = [&](int w) -> uint32_t {
        const int64_t c0 = (int64_t)w * WIN, c1 = (c0 + WIN) < p ? (c0 + WIN) : p;
        return (uint32_t)(((c1 - c0) * (int64_t)sizeof(T)) & ~(int64_t)15);
    };
    // one thread: start the copy of window w into its buffer (a window without a whole 16-byte piece has none)
    auto issue = [&](int w) {
        const uint32_t bytes = bulk_bytes(w);
        if (bytes == 0) return;
        const uint32_t bar = bar0 + 8 * (w % kWinBufs);
        expect_tx(bar, bytes);
        bulk_copy(buf0 + (uint32_t)(w % kWinBufs) * kWinBytes, row + (int64_t)w * WIN, bytes, bar);
    };
    if (tid == 0) {
        for (int b = 0; b <= kWinBufs; ++b) tc::mbar_init(bar0 + 8 * b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (idx_bulk > 0) {
            expect_tx(bar_idx, idx_bulk);
            bulk_copy(tc::smem_u32(sidx), idx, idx_bulk, bar_idx);
        }
        for (int w = 0; w < kWinBufs && w < nwin; ++w) issue(w);
    }
    for (uint32_t b = tid; b < k; b += kRowsThreads) bins[b] = 0.0f;
    for (int64_t j = idx_bulk / 4 + tid; j < kprime; j += kRowsThreads) sidx[j] = __ldg(idx + j);   // at most 3 entries
    __syncthreads();          // barriers initialised, bins zeroed, tail of the index list in place
    bool timed_out = false;
    if (idx_bulk > 0) timed_out = !tc::mbar_wait(bar_idx, 0);
    // where the windows begin in the mask.  The last window takes every remaining position, so that an index
    // >= p is met (and flagged) rather than silently dropped.  (After an expired wait the list may be incomplete:
    // every position then lies in the first window and is checked against it like any other.)
    for (int w = warp; w <= nwin; w += kRowsWarps) {
        int64_t j = w == 0 ? 0 : kprime;
        if (w > 0 && w < nwin && !timed_out) j = warp_lower_bound(sidx, kprime, (uint64_t)w * (uint64_t)WIN);
        if (lane == 0) jb[w] = j;
    }
    __syncthreads();          // window positions known

    bool bad = false;
    float* myq_val = qval + warp * kQueue;
    uint32_t* myq_pos = qpos + warp * kQueue;
    for (int w = 0; w < nwin; ++w) {
        const int64_t c0 = (int64_t)w * WIN, c1 = (c0 + WIN) < p ? (c0 + WIN) : p;
        const int64_t bulk_elems = bulk_bytes(w) / sizeof(T);
        const T* win = reinterpret_cast<const T*>(smem + (size_t)(w % kWinBufs) * kWinBytes);
        const int64_t jlo = jb[w], jhi = jb[w + 1];
        // the window has landed (bounded wait: on expiry its elements count as zeros and the call is flagged)
        bool landed = true;
        if (bulk_elems > 0) landed = tc::mbar_wait(bar0 + 8 * (w % kWinBufs), (uint32_t)(w / kWinBufs) & 1u);
        timed_out = timed_out || !landed;
        // rounds of kRowsThreads * kRowsU positions; the trip count is the same for every thread of a warp
        for (int64_t r0 = jlo; r0 < jhi; r0 += (int64_t)kRowsThreads * kRowsU) {
            float v[kRowsU];
            uint32_t cnt = 0;
#pragma unroll
            for (int u = 0; u < kRowsU; ++u) {
                const int64_t j = r0 + (int64_t)u * kRowsThreads + tid;
                v[u] = 0.0f;
                if (j < jhi) {
                    const int64_t c = (int64_t)sidx[j];
                    if (c < c0 || c >= c1) bad = true;              // not ascending, or >= p: skipped and flagged
                    else if (c - c0 < bulk_elems) v[u] = landed ? elem_value(win[c - c0]) : 0.0f;
                    else v[u] = elem<T>::load(row + c);
                }
                cnt += v[u] != 0.0f ? 1u : 0u;
            }
            // the warp's non-zero entries of this round, compacted: (value, position)
            uint32_t incl = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (lane >= d) incl += t;
            }
            const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);
            uint32_t at = incl - cnt;
#pragma unroll
            for (int u = 0; u < kRowsU; ++u)
                if (v[u] != 0.0f) {
                    myq_val[at] = v[u];
                    myq_pos[at] = (uint32_t)(r0 + (int64_t)u * kRowsThreads + tid);   // < kprime < 2^32
                    ++at;
                }
            __syncwarp();
            for (uint32_t q = lane; q < total; q += 32) {
                const float x = myq_val[q];
                const uint64_t j = (uint64_t)myq_pos[q];
                const uint32_t draws = S1 ? 1u : s;
                for (uint32_t d = 0; d < draws; ++d) {
                    const uint64_t h = sjlt_hash_counter(seed, S1 ? (j + 1) : (j * s + d + 1));
                    const float sx = S1 ? sjlt_signed(h, x) : sjlt_signed(h, x) * scale;
                    atomicAdd(&bins[sjlt_bucket(h, k)], sx);
                }
            }
            __syncwarp();     // the queue is rewritten in the next round
        }
        __syncthreads();      // every thread is done with this buffer: it may be refilled
        if (tid == 0 && w + kWinBufs < nwin) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue(w + kWinBufs);
        }
    }
    if (bad && dev_status) atomicOr(dev_status, GRASS_DEV_BAD_INDEX);
    if (timed_out) {
        // no copy of this block may still be in flight when it leaves: one more bounded wait per barrier
        if (tid == 0) {
            if (dev_status) atomicOr(dev_status, GRASS_DEV_TIMEOUT);
            if (idx_bulk > 0) tc::mbar_wait(bar_idx, 0);
            for (int w = nwin > kWinBufs ? nwin - kWinBufs : 0; w < nwin; ++w)
                if (bulk_bytes(w) > 0) tc::mbar_wait(bar0 + 8 * (w % kWinBufs), (uint32_t)(w / kWinBufs) & 1u);
        }
        __syncthreads();
    }
    for (uint32_t b = tid; b < k; b += kRowsThreads) store_out(out, i * ld_out + b, bins[b], out_bf16);
}

static size_t rows_smem_bytes(int64_t kprime, uint32_t k, uint32_t* idx_bytes)
{
    *idx_bytes = (uint32_t)((kprime * 4 + 15) / 16 * 16);
    return (size_t)kWinBufs * kWinBytes + *idx_bytes + ((size_t)k + 3) / 4 * 4 * sizeof(float) +
           (size_t)kRowsWarps * kQueue * (sizeof(float) + sizeof(uint32_t));
}

bool compress_rows_fits(const void* g, size_t elem_bytes, int64_t p, int64_t ld, const uint32_t* idx, int64_t kprime,
                        uint32_t k, int64_t n)
{
    if (!idx || kprime <= 0 || n <= 0 || n > 0x7FFFFFFFLL) return false;
    if ((uintptr_t)g % 16 != 0 || ((size_t)ld * elem_bytes) % 16 != 0 || (uintptr_t)idx % 16 != 0) return false;
    const int64_t win = kWinBytes / (int64_t)elem_bytes;
    if ((p + win - 1) / win > kMaxWins || kprime * 4 > kMaxIdxBytes) return false;
    uint32_t idx_bytes;
    return rows_smem_bytes(kprime, k, &idx_bytes) <= 110 * 1024;    // two thread blocks per SM
}

template <typename T>
static grass_status launch_rows_t(const T* g, int64_t n, int64_t p, int64_t ld, const uint32_t* idx, int64_t kprime,
                                  const grass_sjlt_spec& sp, float* out, int64_t ld_out, uint32_t* dev_status,
                                  cudaStream_t st, int out_bf16)
{
    uint32_t idx_bytes = 0;
    const size_t smem = rows_smem_bytes(kprime, sp.k, &idx_bytes);
    const float scale = 1.0f / sqrtf((float)sp.s);
    auto launch = [&](auto kern) -> grass_status {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return GRASS_ERR_CUDA;
        kern<<<dim3((unsigned)n, 1, 1), kRowsThreads, smem, st>>>(g, p, ld, idx, kprime, sp.k, sp.s, sp.seed, scale, out,
                                                                  ld_out, idx_bytes, dev_status, out_bf16);
        return launch_status();
    };
    if (sp.s == 1) return launch(grass_compress_rows_kernel<T, true>);
    return launch(grass_compress_rows_kernel<T, false>);
}

grass_status launch_compress_rows(const void* g, grass_dtype dt, int64_t n, int64_t p, int64_t ld, const uint32_t* idx,
                                  int64_t kprime, const grass_sjlt_spec& sp, float* out, int64_t ld_out,
                                  uint32_t* dev_status, cudaStream_t st, int out_bf16)
{
    if (dt == GRASS_F32)
        return launch_rows_t<float>((const float*)g, n, p, ld, idx, kprime, sp, out, ld_out, dev_status, st, out_bf16);
    return launch_rows_t<__nv_bfloat16>((const __nv_bfloat16*)g, n, p, ld, idx, kprime, sp, out, ld_out, dev_status, st,
                                        out_bf16);
}

}  // namespace grass
