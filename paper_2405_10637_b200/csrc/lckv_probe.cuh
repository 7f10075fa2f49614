// Read-only streaming probes: how fast can this GPU read device memory when nothing else is done
// with the bytes?  The decode attention kernels are read-dominated, so their ceiling is a read
// stream, not the read + write copy that bandwidth figures are usually quoted from.
//   kind 0: every thread issues independent 16-byte loads (grid-stride, 8 in flight per thread) and
//           folds them into a checksum;
//   kind 2: the same with 32-byte loads marked evict-first in L2;
//   (every kind can pass over the buffer several times in one launch: with a buffer that fits the L2
//   the later passes measure the L2's read bandwidth instead of the memory's)
//   kind 1: every warp moves 8 KB pieces into its own shared-memory ring with 1-D bulk copies, the way
//           the attention kernels stream K and V, and reads one word of each piece.
#pragma once
#include "lckv_device.cuh"

namespace lckv {

constexpr int kProbeThreads = 256;
constexpr int kProbeWarps = kProbeThreads / 32;
constexpr int kProbeSlots = 2;
constexpr int kProbePiece = 8192;
constexpr int kProbeSmemBytes = kProbeWarps * kProbeSlots * (kProbePiece + 8);

__device__ __forceinline__ uint4 ldg_stream16(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 32-byte load (sm_100), marked evict-first in L2; p must be 32-byte aligned.  Returns the word sum.
__device__ __forceinline__ uint32_t ldg_stream32_sum(const void* p)
{
    uint32_t a, b, c, d, e, f, g, h;
    asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(a), "=r"(b), "=r"(c), "=r"(d), "=r"(e), "=r"(f), "=r"(g), "=r"(h)
                 : "l"(p));
    return a + b + c + d + e + f + g + h;
}

// n16 = number of 16-byte words.  sum receives the wrapped 32-bit sum of all 32-bit words read.
__global__ void __launch_bounds__(kProbeThreads) read_stream_ldg_kernel(const uint4* __restrict__ src,
                                                                        uint64_t n16, uint32_t* sum,
                                                                        int repeats)
{
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    uint32_t acc = 0;
    for (int rep = 0; rep < repeats; ++rep) {
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 7 * stride < n16; i += 8 * stride) {
        uint4 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = ldg_stream16(src + i + k * stride);
#pragma unroll
        for (int k = 0; k < 8; ++k) acc += v[k].x + v[k].y + v[k].z + v[k].w;
    }
    for (; i < n16; i += stride) {
        const uint4 v = ldg_stream16(src + i);
        acc += v.x + v.y + v.z + v.w;
    }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if ((threadIdx.x & 31) == 0) atomicAdd(sum, acc);
}

// The same with 32-byte loads: n32 = number of 32-byte words.
__global__ void __launch_bounds__(kProbeThreads) read_stream_ldg32_kernel(const uint8_t* __restrict__ src,
                                                                          uint64_t n32, uint32_t* sum,
                                                                          int repeats)
{
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    uint32_t acc = 0;
    for (int rep = 0; rep < repeats; ++rep) {
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n32; i += 4 * stride) {
        uint32_t v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = ldg_stream32_sum(src + (i + k * stride) * 32);
        acc += v[0] + v[1] + v[2] + v[3];
    }
    for (; i < n32; i += stride) acc += ldg_stream32_sum(src + i * 32);
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if ((threadIdx.x & 31) == 0) atomicAdd(sum, acc);
}

// n_pieces pieces of kProbePiece bytes; piece i goes to warp i % (all warps).  sum receives the sum of
// the first word of every piece.  Waits are bounded; a wait that runs out sets *status.
__global__ void __launch_bounds__(kProbeThreads, 1) read_stream_bulk_kernel(const uint8_t* __restrict__ src,
                                                                            uint64_t n_pieces, uint32_t* sum,
                                                                            int32_t* status, int repeats,
                                                                            float l2_keep)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint64_t n_warps = (uint64_t)gridDim.x * kProbeWarps;
    const uint64_t w = (uint64_t)blockIdx.x * kProbeWarps + warp;
    const uint32_t ring = smem_u32(smem) + warp * (kProbeSlots * kProbePiece);
    const uint32_t bars = smem_u32(smem) + kProbeWarps * kProbeSlots * kProbePiece + warp * (kProbeSlots * 8);
    if (lane == 0) {
        for (int s = 0; s < kProbeSlots; ++s) mbar_init(bars + 8 * s, 1);
        fence_mbar_init();
    }
    __syncwarp();
    // contiguous range per warp, like a worker's run of tiles
    const uint64_t lo0 = w * n_pieces / n_warps, per = (w + 1) * n_pieces / n_warps - lo0;
    // `repeats` passes over the warp's range, as one run of pieces: piece index i reads lo0 + i % per
    const uint64_t lo = 0, hi = per * (uint64_t)repeats;
    const uint64_t pol = make_l2_policy(l2_keep);
    uint64_t issued = lo;
    uint32_t islot = 0, cslot = 0, cphase = 0, acc = 0;
    bool ok = true;
    auto issue = [&]() {
        if (lane == 0) {
            mbar_expect_tx(bars + 8 * islot, kProbePiece);
            bulk_g2s_hint(ring + islot * kProbePiece, src + (lo0 + issued % per) * kProbePiece, kProbePiece,
                          bars + 8 * islot, pol);
        }
        ++issued;
        islot = (islot + 1 == kProbeSlots) ? 0 : islot + 1;
    };
    while (issued < hi && issued < lo + kProbeSlots) issue();
    for (uint64_t i = lo; i < hi; ++i) {
        if (!mbar_wait_bounded(bars + 8 * cslot, cphase)) { ok = false; break; }
        if (lane == 0) acc += lds128(ring + cslot * kProbePiece).x;
        __syncwarp();
        if (issued < hi) issue();
        cslot = (cslot + 1 == kProbeSlots) ? 0 : cslot + 1;
        if (cslot == 0) cphase ^= 1;
    }
    if (lane == 0 && per) atomicAdd(sum, acc);
    if (!ok) {
        if (lane == 0) atomicExch(status, kStatusTimeout);
        for (int s = 0; s < kProbeSlots; ++s) {
            mbar_wait_bounded(bars + 8 * s, 0, 1u << 10);
            mbar_wait_bounded(bars + 8 * s, 1, 1u << 10);
        }
    }
}

}  // namespace lckv
