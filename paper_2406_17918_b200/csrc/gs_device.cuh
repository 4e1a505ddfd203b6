// Device-side primitives: Philox4x32-10, warp selection, block scan.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gs {

constexpr uint32_t FULL = 0xFFFFFFFFu;
constexpr int CAND_CAP = 128;  // candidate buffer entries per node (4 per lane)

enum Purpose : uint32_t { FILL = 1, EVICT = 2, PICK = 3 };

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and a key bump.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Same function with the ten round keys precomputed (k0 + i*0x9E3779B9, k1 + i*0xBB67AE85): when
// `rk` lives in kernel-parameter space the keys become constant-bank operands of the xors.
__device__ __forceinline__ uint4 philox4x32_10_rk(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                  const uint32_t (&rk)[20]) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ rk[2 * round];
        const uint32_t n2 = hi0 ^ c3 ^ rk[2 * round + 1];
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    }
    return make_uint4(c0, c1, c2, c3);
}

// The same function for the consecutive quads of one row, as the threshold scan evaluates it: counter
// (q, node, step, word) with only q changing.  The first round's products are then M1 * step (one value per
// launch) and M0 * q (which grows by a constant from quad to quad: a 64-bit add instead of a multiply), and
// in the second round M0 multiplies a value that depends on the node alone (once per row).  What is left per
// block are 17 wide multiplies instead of 20; the result is the same word for word.
struct RowKeys {
    uint32_t cw;    // word ^ rk[1]
    uint32_t d;     // lo(M1 * step) ^ rk[2]
    uint32_t b;     // hi(M0 * a) ^ rk[3], a = hi(M1 * step) ^ node ^ rk[0]
    uint32_t lo_a;  // lo(M0 * a)
};
constexpr uint32_t PHILOX_M0 = 0xD2511F53u, PHILOX_M1 = 0xCD9E8D57u;

__device__ __forceinline__ RowKeys philox_row_keys(uint32_t node, uint32_t step, uint32_t word, const uint32_t (&rk)[20]) {
    const uint32_t a = __umulhi(PHILOX_M1, step) ^ node ^ rk[0];
    RowKeys k;
    k.cw = word ^ rk[1];
    k.d = (PHILOX_M1 * step) ^ rk[2];
    k.b = __umulhi(PHILOX_M0, a) ^ rk[3];
    k.lo_a = PHILOX_M0 * a;
    return k;
}

// a + b on the integer adder (add with carry), so that it does not compete with the multiplies for their pipe
__device__ __forceinline__ unsigned long long add64(unsigned long long a, unsigned long long b) {
    uint32_t lo, hi;
    asm("add.cc.u32 %0, %2, %4;\n\taddc.u32 %1, %3, %5;"
        : "=r"(lo), "=r"(hi)
        : "r"((uint32_t)a), "r"((uint32_t)(a >> 32)), "r"((uint32_t)b), "r"((uint32_t)(b >> 32)));
    return ((unsigned long long)hi << 32) | lo;
}

// p0 = M0 * q as a 64-bit product; the block of quad q + j is philox_row_block(p0 + j * M0, ...).
__device__ __forceinline__ uint4 philox_row_block(unsigned long long p0, const RowKeys& k, const uint32_t (&rk)[20]) {
    const uint32_t x = (uint32_t)(p0 >> 32) ^ k.cw;                 // third counter word after round one
    uint32_t c0 = __umulhi(PHILOX_M1, x) ^ k.d, c1 = PHILOX_M1 * x;   // round two
    uint32_t c2 = k.b ^ (uint32_t)p0, c3 = k.lo_a;
#pragma unroll
    for (int round = 2; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(PHILOX_M0, c0), lo0 = PHILOX_M0 * c0;
        const uint32_t hi1 = __umulhi(PHILOX_M1, c2), lo1 = PHILOX_M1 * c2;
        const uint32_t n0 = hi1 ^ c1 ^ rk[2 * round];
        const uint32_t n2 = hi0 ^ c3 ^ rk[2 * round + 1];
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Kernels of a batch are launched with programmatic stream serialization: a kernel may be set up on the GPU
// while its predecessor in the stream is still draining, and must call this before it reads anything the
// predecessor wrote (it returns once the predecessor has completed and its writes are visible).
__device__ __forceinline__ void chain_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ uint32_t word_of(const uint4& o, uint32_t w) {
    return w == 0 ? o.x : (w == 1 ? o.y : (w == 2 ? o.z : o.w));
}

__device__ __forceinline__ uint32_t lanemask_lt() {
    uint32_t m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// Lanes in `valid` hold (key, lane) pairs; returns the mask of the k pairs smallest in
// (key, lane) order.  Keys are uniform 32-bit words, so the lanes with key <= k/n * 2^32 are
// already close to the answer; the difference is repaired by a few rounds of a warp-wide max
// (drop the largest selected pair) or min (add the smallest unselected pair).  Any guess gives
// the exact result: every selected key is <= every unselected key.
__device__ __forceinline__ uint32_t warp_smallest_k(uint32_t key, uint32_t valid, int k, int lane) {
    const int n = __popc(valid);
    if (k >= n) return valid;
    if (k <= 0) return 0u;
    const bool mine = (valid >> lane) & 1u;
    const uint32_t guess = __float2uint_rz(__fdividef((float)k, (float)n) * 4294967040.0f);  // k < n <= 32
    uint32_t sel = __ballot_sync(FULL, mine && key <= guess);
    int c = __popc(sel);
    while (c > k) {   // drop the largest selected pair: max key, highest lane among equals
        const bool live = (sel >> lane) & 1u;
        const uint32_t x = live ? key : 0u;
        const uint32_t m = __reduce_max_sync(FULL, x);
        const uint32_t b = __ballot_sync(FULL, live && x == m);
        sel &= ~(0x80000000u >> __clz(b));
        --c;
    }
    while (c < k) {   // add the smallest unselected pair: min key, lowest lane among equals
        const bool live = mine && !((sel >> lane) & 1u);
        const uint32_t x = live ? key : 0xFFFFFFFFu;
        const uint32_t m = __reduce_min_sync(FULL, x);
        const uint32_t b = __ballot_sync(FULL, live && x == m);
        sel |= b & (0u - b);
        ++c;
    }
    return sel;
}

// Exclusive scan of one int per thread over a block of BT threads (BT a multiple of 32, <= 1024).
// `warp_sums` is shared memory with at least 33 ints.  Returns the exclusive prefix; *total gets
// the block sum.  Contains __syncthreads: every thread of the block must call it.
template <int BT>
__device__ __forceinline__ int block_exclusive_scan(int x, int* warp_sums, int* total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(FULL, incl, d);
        if (lane >= d) incl += y;
    }
    __syncthreads();  // protects warp_sums against a previous call's readers
    if (lane == 31) warp_sums[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        int s = (lane < BT / 32) ? warp_sums[lane] : 0;
        int si = s;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(FULL, si, d);
            if (lane >= d) si += y;
        }
        if (lane < BT / 32) warp_sums[lane] = si - s;
        if (lane == 31) warp_sums[32] = si;
    }
    __syncthreads();
    *total = warp_sums[32];
    return warp_sums[wid] + incl - x;
}

// In-place exclusive scan of tile_sums[0..T) by one block of BT threads; returns the total.
template <int BT>
__device__ __forceinline__ int scan_tiles_in_place(int32_t* tile_sums, int T, int* warp_sums) {
    int carry = 0;
    for (int base = 0; base < T; base += BT) {
        const int i = base + (int)threadIdx.x;
        const int x = (i < T) ? __ldcg(tile_sums + i) : 0;
        int total;
        const int excl = block_exclusive_scan<BT>(x, warp_sums, &total);
        if (i < T) tile_sums[i] = carry + excl;
        carry += total;
    }
    return carry;
}

__device__ __forceinline__ void raise_status(int32_t* status, int code) { atomicCAS(status, 0, code); }

}  // namespace gs
