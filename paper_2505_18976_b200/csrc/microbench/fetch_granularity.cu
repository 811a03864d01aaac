// Microbenchmark behind the roofline denominator of the gather kernels: how many bytes does HBM
// deliver per 4-byte read when reads are `stride` bytes apart, for several load flavours
// (read-only ld, L2-coherent ld, 16-byte vector ld, the L2 prefetch-size hints, cp.async, 16/32-byte
// bulk-copy engine transfers)?
// Run plain for reads/s; run under `ncu --metrics dram__bytes_read.sum` for bytes per read.
// Every wait on an mbarrier is bounded and the kernel leaves with a flag set if one expires.
#include <cstdio>
#include <cstdint>
#include <cstdlib>
#include <cuda_runtime.h>
#define CK(x) do{cudaError_t e=(x); if(e!=cudaSuccess){printf("err %s line %d\n", cudaGetErrorString(e), __LINE__); return 1;}}while(0)

template <int MODE>
__global__ void rd(const uint32_t* __restrict__ p, size_t n_reads, size_t stride_words, uint32_t* out)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t acc = 0;
    for (; i < n_reads; i += (size_t)gridDim.x * blockDim.x) {
        const uint32_t* q = p + i * stride_words;
        uint32_t v;
        if (MODE == 0) v = __ldg(q);
        else if (MODE == 1) asm volatile("ld.relaxed.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 2) asm volatile("ld.volatile.global.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 3) asm volatile("ld.global.cv.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 4) asm volatile("ld.global.L1::no_allocate.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 5) asm volatile("ld.relaxed.sys.global.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 6) { uint4 w; asm volatile("ld.global.nc.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w.x),"=r"(w.y),"=r"(w.z),"=r"(w.w) : "l"(q)); v = w.x ^ w.y ^ w.z ^ w.w; }
        // the documented L2 prefetch-size hints, and a 2-byte load as the gather kernels issue
        else if (MODE == 7) asm volatile("ld.global.L2::64B.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 8) asm volatile("ld.global.L2::128B.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 9) asm volatile("ld.global.nc.L1::no_allocate.L2::64B.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 10) asm volatile("ld.global.L2::256B.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 11) { uint16_t h; asm volatile("ld.global.nc.b16 %0, [%1];" : "=h"(h) : "l"(q)); v = h; }
        // the 64-byte hint on loads that bypass L1
        else if (MODE == 12) asm volatile("ld.global.cg.L2::64B.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else if (MODE == 13) asm volatile("ld.relaxed.gpu.global.L2::64B.b32 %0, [%1];" : "=r"(v) : "l"(q));
        else asm volatile("ld.global.cs.L2::64B.b32 %0, [%1];" : "=r"(v) : "l"(q));
        acc ^= v;
    }
    // a value the loaded data can produce for no mode, so the store never happens but cannot be proven dead
    if (acc == (MODE == 11 ? 0x5678u : 0x12345678u)) out[0] = acc;
}

// cp.async (the non-bulk asynchronous copy) of BYTES = 4 (through L1) or 16 (L2 only, optionally with the
// 64-byte prefetch-size hint) into a per-thread shared-memory slot
template <int BYTES, bool HINT64>
__global__ void rd_cp_async(const uint32_t* __restrict__ p, size_t n_reads, size_t stride_words, uint32_t* out)
{
    __shared__ __align__(16) uint32_t slot[4][256 * 4];          // four destinations per thread, used in turn
    const uint32_t dst0 = (uint32_t)__cvta_generic_to_shared(&slot[0][threadIdx.x * 4]);
    slot[0][threadIdx.x * 4] = 0;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t turn = 0;
    for (; i < n_reads; i += (size_t)gridDim.x * blockDim.x, ++turn) {
        const uint32_t* q = p + i * stride_words;
        const uint32_t dst = dst0 + (turn & 3u) * (uint32_t)sizeof(slot[0]);
        if (BYTES == 4) asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(q) : "memory");
        else if (HINT64) asm volatile("cp.async.cg.shared.global.L2::64B [%0], [%1], 16;" ::"r"(dst), "l"(q) : "memory");
        else asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(q) : "memory");
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (slot[0][threadIdx.x * 4] == 0x12345678u) out[0] = 1;
}

// bulk (TMA) 1D copies of BYTES each, one per thread of warp 0..., completion on an mbarrier
template <int BYTES>
__global__ void rd_bulk(const uint32_t* __restrict__ p, size_t n_reads, size_t stride_words, uint32_t* out)
{
    __shared__ __align__(128) unsigned char buf[128 * 32];
    __shared__ __align__(8) unsigned long long bar;
    const int tid = threadIdx.x;
    uint32_t bar_a = (uint32_t)__cvta_generic_to_shared(&bar);
    if (tid == 0) { asm volatile("mbarrier.init.shared.b64 [%0], 1;" :: "r"(bar_a)); }
    __syncthreads();
    uint32_t phase = 0, acc = 0;
    const size_t per_iter = blockDim.x;
    for (size_t base = (size_t)blockIdx.x * per_iter; base < n_reads; base += (size_t)gridDim.x * per_iter) {
        size_t i = base + tid;
        if (tid == 0) {
            size_t cnt = (n_reads - base) < per_iter ? (n_reads - base) : per_iter;
            asm volatile("mbarrier.arrive.expect_tx.shared.b64 _, [%0], %1;" :: "r"(bar_a), "r"((uint32_t)(cnt * BYTES)));
        }
        __syncthreads();
        if (i < n_reads) {
            uint32_t dst = (uint32_t)__cvta_generic_to_shared(buf + tid * BYTES);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         :: "r"(dst), "l"(p + i * stride_words), "r"(BYTES), "r"(bar_a) : "memory");
        }
        // bounded wait
        uint32_t done = 0; int spins = 0;
        while (!done && spins < 2000000) {
            asm volatile("{ .reg .pred P; mbarrier.try_wait.parity.shared.b64 P, [%1], %2; selp.u32 %0, 1, 0, P; }" : "=r"(done) : "r"(bar_a), "r"(phase));
            ++spins;
        }
        if (__syncthreads_or(!done)) { if (tid == 0) out[1] = 0xDEAD; break; }
        phase ^= 1;
        acc ^= *reinterpret_cast<uint32_t*>(buf + tid * BYTES);
        __syncthreads();
    }
    if (acc == 0x12345678u) out[0] = acc;
}

int main(int argc, char** argv)
{
    // optional argument: value for cudaLimitMaxL2FetchGranularity (32, 64 or 128), set before anything
    // else touches the device; the value the driver reports back is printed
    if (argc > 1) {
        CK(cudaDeviceSetLimit(cudaLimitMaxL2FetchGranularity, (size_t)atoi(argv[1])));
    }
    size_t gran = 0;
    CK(cudaDeviceGetLimit(&gran, cudaLimitMaxL2FetchGranularity));
    printf("cudaLimitMaxL2FetchGranularity = %zu\n", gran);
    const size_t bytes = 2ull << 30;
    uint32_t *p, *out;
    CK(cudaMalloc(&p, bytes)); CK(cudaMemset(p, 1, bytes)); CK(cudaMalloc(&out, 64)); CK(cudaMemset(out, 0, 64));
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    const size_t strides[] = {32, 64, 128, 256, 512};
    for (size_t sb : strides) {
        size_t n_reads = bytes / sb;
        if (n_reads > (1ull << 24)) n_reads = 1ull << 24;   // 16M reads
        auto run = [&](auto kern, const char* name, int threads) {
            kern<<<148 * 8, threads>>>(p, n_reads, sb / 4, out);
            cudaEventRecord(e0);
            kern<<<148 * 8, threads>>>(p, n_reads, sb / 4, out);
            cudaEventRecord(e1); cudaEventSynchronize(e1);
            float ms; cudaEventElapsedTime(&ms, e0, e1);
            printf("%-14s stride %4zu B: %8.1f us  %7.1f Greads/s\n", name, sb, ms * 1e3, n_reads / ms * 1e-6);
            return 0;
        };
        run(rd<0>, "ldg", 256); run(rd<1>, "relaxed.gpu", 256); run(rd<2>, "volatile", 256); run(rd<3>, "cv", 256);
        run(rd<4>, "no_allocate", 256); run(rd<5>, "relaxed.sys", 256); run(rd<6>, "nc.v4", 256);
        run(rd<7>, "L2::64B", 256); run(rd<8>, "L2::128B", 256); run(rd<9>, "nc.noalloc.64B", 256);
        run(rd<10>, "L2::256B", 256); run(rd<11>, "nc.b16", 256);
        run(rd<12>, "cg.64B", 256); run(rd<13>, "relaxed.gpu.64B", 256); run(rd<14>, "cs.64B", 256);
        run(rd_cp_async<4, false>, "cp.async.ca4", 256); run(rd_cp_async<16, false>, "cp.async.cg16", 256);
        run(rd_cp_async<16, true>, "cp.async.cg16.64B", 256);
        run(rd_bulk<16>, "bulk16", 128); run(rd_bulk<32>, "bulk32", 128);
    }
    uint32_t h[2]; CK(cudaMemcpy(h, out, 8, cudaMemcpyDeviceToHost));
    printf("flags %x %x\n", h[0], h[1]);
    CK(cudaDeviceSynchronize());
    return 0;
}
