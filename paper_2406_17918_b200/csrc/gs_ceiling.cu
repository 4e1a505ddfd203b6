// Measured integer-ALU ceilings of the key function: how many Philox4x32-10 blocks, 32x32->64
// multiplies and three-input logic operations per second this GPU sustains when a kernel does
// nothing else.  The threshold scan of the sampler is bound by exactly this arithmetic, so these
// figures are the roofline it is reported against.  Nothing here is on the sampling path.
#include "gs_device.cuh"
#include "gs_internal.h"

namespace gs {

__device__ unsigned int g_ceiling_sink;

constexpr int CEIL_THREADS = 256;

// Philox blocks with the scan's threshold test: four independent blocks per thread and iteration,
// counters that change every iteration, one warp vote per iteration - the inner loop of the scan
// without any of its bookkeeping, in the scan's form of the function (consecutive quads of one row:
// 17 wide multiplies per block).  `tinc` is a run-time value no key ever meets, so nothing is stored.
__global__ void __launch_bounds__(CEIL_THREADS) k_ceiling_philox(const __grid_constant__ StepParams P, int iters,
                                                                   uint32_t tinc) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t v = blockIdx.x * CEIL_THREADS + threadIdx.x;
    uint32_t found = 0;
    const RowKeys rkeys = philox_row_keys(v, P.step, P.word_fill, P.rk);
    constexpr unsigned long long M0x32 = 32ull * PHILOX_M0;
    unsigned long long p0 = (unsigned long long)PHILOX_M0 * lane;
    for (int it = 0; it < iters; ++it, p0 = add64(p0, 4 * M0x32)) {
        const uint4 o0 = philox_row_block(p0, rkeys, P.rk);
        const uint4 o1 = philox_row_block(add64(p0, M0x32), rkeys, P.rk);
        const uint4 o2 = philox_row_block(add64(p0, 2 * M0x32), rkeys, P.rk);
        const uint4 o3 = philox_row_block(add64(p0, 3 * M0x32), rkeys, P.rk);
        const uint32_t m0 = __vimin3_u32(o0.x, o0.y, o0.z), m1 = __vimin3_u32(o1.x, o1.y, o1.z);
        const uint32_t m2 = __vimin3_u32(o2.x, o2.y, o2.z), m3 = __vimin3_u32(o3.x, o3.y, o3.z);
        const uint32_t ma = __vimin3_u32(m0, o0.w, o1.w), mb = __vimin3_u32(m1, o2.w, o3.w);
        if (__ballot_sync(FULL, min(__vimin3_u32(ma, mb, m2), m3) < tinc) == 0) continue;
        found += 1;
    }
    if (found) atomicAdd(&g_ceiling_sink, found);
}

// Eight independent chains of x <- lo(M*x) ^ hi(M*x): one wide multiply and one logic operation per step.
__global__ void __launch_bounds__(CEIL_THREADS) k_ceiling_mul(int iters, uint32_t seed, uint32_t never) {
    uint32_t x[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) x[j] = seed + blockIdx.x * CEIL_THREADS + threadIdx.x + 0x9E3779B9u * j;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t m = (j & 1) ? 0xCD9E8D57u : 0xD2511F53u;
            x[j] = __umulhi(m, x[j]) ^ (m * x[j]);
        }
    }
    uint32_t acc = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) acc ^= x[j];
    if (acc == never) atomicAdd(&g_ceiling_sink, 1u);
}

// Eight independent chains of three-input logic operations (a <- (a & b) ^ c style, not reducible).
__global__ void __launch_bounds__(CEIL_THREADS) k_ceiling_logic(int iters, uint32_t seed, uint32_t never) {
    uint32_t a[8], b[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        a[j] = seed + blockIdx.x * CEIL_THREADS + threadIdx.x + 0x9E3779B9u * j;
        b[j] = ~a[j] * 3u;
    }
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t r;
            // (a & b) ^ c with c = the neighbouring chain's value: lookup table 0x78 = (a & b) ^ c
            asm volatile("lop3.b32 %0, %1, %2, %3, 0x78;" : "=r"(r) : "r"(a[j]), "r"(b[j]), "r"(a[(j + 1) & 7]));
            b[j] = a[j];
            a[j] = r;
        }
    }
    uint32_t acc = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) acc ^= a[j] ^ b[j];
    if (acc == never) atomicAdd(&g_ceiling_sink, 1u);
}

}  // namespace gs

using namespace gs;

extern "C" gs_status gs_alu_ceiling(int32_t what, int32_t milliseconds, void* stream, double* h_units_per_second) {
    if (!h_units_per_second) return set_error(GS_ERR_ARG, "h_units_per_second is NULL");
    if (what < 0 || what > 2) return set_error(GS_ERR_ARG, "what %d outside [0, 2]", what);
    if (milliseconds < 1 || milliseconds > 2000) return set_error(GS_ERR_ARG, "milliseconds outside [1, 2000]");
    cudaStream_t s = (cudaStream_t)stream;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e != cudaSuccess) {
        if (e0) cudaEventDestroy(e0);
        return set_error(GS_ERR_CUDA, "cudaEventCreate: %s", cudaGetErrorString(e));
    }
    StepParams P{};
    P.step = 1;
    P.word_fill = (1u << 8);
    for (int i = 0; i < 10; ++i) {
        P.rk[2 * i] = 0xF3BCC908u + (uint32_t)i * 0x9E3779B9u;
        P.rk[2 * i + 1] = 0x6A09E667u + (uint32_t)i * 0xBB67AE85u;
    }
    const int grid = (int)(sm_count() * 8);
    // units one thread evaluates per iteration
    const double per_iter = what == 0 ? 4.0 : 8.0;
    int iters = 256;
    double rate = 0.0;
    // the first launch sizes the timed one (and warms the clocks up): aim at `milliseconds` of work
    for (int pass = 0; pass < 3; ++pass) {
        cudaEventRecord(e0, s);
        if (what == 0) k_ceiling_philox<<<grid, CEIL_THREADS, 0, s>>>(P, iters, 0u);
        else if (what == 1) k_ceiling_mul<<<grid, CEIL_THREADS, 0, s>>>(iters, 12345u, 0u);
        else k_ceiling_logic<<<grid, CEIL_THREADS, 0, s>>>(iters, 12345u, 0u);
        count_launches(1);
        e = cudaGetLastError();
        cudaEventRecord(e1, s);
        if (e == cudaSuccess) e = cudaEventSynchronize(e1);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
        if (e != cudaSuccess) break;
        rate = per_iter * (double)iters * (double)grid * CEIL_THREADS / ((double)ms * 1e-3);
        if (pass < 2) {
            double want = (double)iters * (double)milliseconds / (ms > 1e-3f ? (double)ms : 1e-3);
            if (pass == 0) want *= 0.25;   // a short second launch, then the timed one
            iters = want > 4.0e6 ? 4000000 : (want < 16.0 ? 16 : (int)want);
        }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) return set_error(GS_ERR_CUDA, "ceiling kernel: %s", cudaGetErrorString(e));
    *h_units_per_second = rate;
    return GS_OK;
}
