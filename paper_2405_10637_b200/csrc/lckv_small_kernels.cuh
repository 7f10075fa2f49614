// Small kernels around the attention kernels: work plan, append, length advance.
#pragma once
#include "lckv_device.cuh"

namespace lckv {

// ---------------------------------------------------------------------------------------------
// Work plan for one decode step.  The attention kernels treat a launch as one long sequence of
// tiles: sequence b contributes ceil(n_vis[b] / R) tiles for each of its H pairs, in the order
// (b, pair, tile), and the sequence is cut into equal contiguous ranges, one per worker warp.
// This kernel (one block) writes, for both mask modes (n_vis = len + mode):
//   pre[mode][b]    tiles of sequences 0..b-1 (exclusive prefix; pre[mode][B] = all tiles / H)
//   start[mode][w]  where worker w's range begins and how long it is, with everything about that
//                   sequence a worker needs to issue its first copy (one 32-byte load, no chain of
//                   dependent look-ups at the start of an attention launch)
// n_vis is capped at T_cap: in streaming mode (sink + recent window) a cache never holds more than
// T_cap rows; a negative length counts as zero rows.
// ---------------------------------------------------------------------------------------------
struct __align__(32) WorkerStart {
    int32_t b, h;        // sequence and pair in which the range begins
    uint32_t t, nt;      // first tile within that pair; tiles per pair of sequence b
    int32_t nv;          // visible rows of sequence b
    uint32_t pre0;       // pre[b]
    uint32_t n_tiles;    // length of the range (0: no work)
    uint32_t pad;
};

__device__ __forceinline__ WorkerStart load_worker_start(const WorkerStart* p)
{
    const uint4 lo = __ldg(reinterpret_cast<const uint4*>(p));
    const uint4 hi = __ldg(reinterpret_cast<const uint4*>(p) + 1);
    WorkerStart s;
    s.b = (int32_t)lo.x; s.h = (int32_t)lo.y; s.t = lo.z; s.nt = lo.w;
    s.nv = (int32_t)hi.x; s.pre0 = hi.y; s.n_tiles = hi.z; s.pad = 0;
    return s;
}

__global__ void __launch_bounds__(1024)
plan_kernel(const int32_t* __restrict__ lens, int B, int R, int H, int n_workers,
            uint32_t* pre, int pre_stride, WorkerStart* __restrict__ start, int T_cap)
{
    __shared__ uint32_t warp_sums[32];
    __shared__ uint32_t carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk = (B + 1023) / 1024;

    for (int mode = 0; mode < 2; ++mode) {
        uint32_t* pr = pre + mode * pre_stride;
        const int b0 = min(B, tid * chunk), b1 = min(B, b0 + chunk);
        uint32_t local = 0;
        for (int b = b0; b < b1; ++b) local += (uint32_t)(visible_rows(lens[b], mode, T_cap) + R - 1) / (uint32_t)R;
        // block-wide exclusive scan of `local`
        uint32_t incl = local;
        for (int off = 1; off < 32; off <<= 1) {
            uint32_t v = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += v;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            uint32_t ws = warp_sums[lane], wi = ws;
            for (int off = 1; off < 32; off <<= 1) {
                uint32_t v = __shfl_up_sync(0xffffffffu, wi, off);
                if (lane >= off) wi += v;
            }
            warp_sums[lane] = wi - ws;  // exclusive prefix of the warp sums
            if (lane == 31) carry = wi;
        }
        __syncthreads();
        uint32_t run = warp_sums[warp] + incl - local;
        for (int b = b0; b < b1; ++b) {
            pr[b] = run;
            run += (uint32_t)(visible_rows(lens[b], mode, T_cap) + R - 1) / (uint32_t)R;
        }
        if (tid == 0) pr[B] = carry;
        __syncthreads();  // pr[] (global) is now visible to the whole block

        const uint64_t total = (uint64_t)carry * (uint64_t)H;
        const uint64_t n_eff = total < (uint64_t)n_workers ? total : (uint64_t)n_workers;
        for (int w = tid; w < n_workers; w += 1024) {
            uint4 s0 = make_uint4(0, 0, 0, 0), s1 = s0;
            if ((uint64_t)w < n_eff) {
                const uint64_t lo = (uint64_t)w * total / n_eff;
                const uint64_t hi = (uint64_t)(w + 1) * total / n_eff;
                const uint32_t x = (uint32_t)(lo / (uint64_t)H);
                // largest b with pre[b] <= x (then pre[b+1] > x)
                int lo_i = 0, hi_i = B;  // invariant: pre[lo_i] <= x < pre[hi_i]
                while (hi_i - lo_i > 1) {
                    const int mid = (lo_i + hi_i) >> 1;
                    if (pr[mid] <= x) lo_i = mid; else hi_i = mid;
                }
                const uint32_t pre0 = pr[lo_i], nt = pr[lo_i + 1] - pre0;
                const uint64_t rel = lo - (uint64_t)pre0 * (uint64_t)H;
                s0 = make_uint4((uint32_t)lo_i, (uint32_t)(rel / nt), (uint32_t)(rel % nt), nt);
                s1 = make_uint4((uint32_t)visible_rows(lens[lo_i], mode, T_cap), pre0, (uint32_t)(hi - lo), 0u);
            }
            uint4* dst = reinterpret_cast<uint4*>(start + (size_t)mode * n_workers + w);
            dst[0] = s0;
            dst[1] = s1;
        }
        __syncthreads();
    }
}

// Row len[b] of K and V <- k_new, v_new (bit-exact 16-byte copies).  One thread per 16 bytes.
// With n_sink > 0 (StreamingLLM-style cache, paper Section 3.3) token t >= T_cap replaces the oldest
// non-sink token: row n_sink + (t - n_sink) mod (T_cap - n_sink).
__global__ void append_kernel(uint16_t* __restrict__ K, uint16_t* __restrict__ V,
                              const uint16_t* __restrict__ k_new,
                              const uint16_t* __restrict__ v_new,
                              const int32_t* __restrict__ lens, int B, int H_kv, int64_t T_cap,
                              int D, int n_sink, const int32_t* __restrict__ page_table,
                              int pt_stride, int page_shift)
{
    const int chunks = D / 8;
    const int64_t n = (int64_t)B * H_kv * chunks;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int c = (int)(i % chunks);
    const int64_t bh = i / chunks;
    const int b = (int)(bh / H_kv);
    int64_t row = lens[b];
    // Streaming mode: the first n_sink rows stay, the others form a ring of the most recent tokens.
    if (n_sink > 0 && row >= T_cap) row = n_sink + (row - n_sink) % (T_cap - n_sink);
    if (row < 0 || row >= T_cap) return;  // the host refuses such calls; never write out of range
    int64_t dst_row = bh * T_cap + row;
    if (page_table) {   // paged slot [n_pages, H_kv, page_rows, D]
        const int64_t id = page_table[(int64_t)b * pt_stride + (row >> page_shift)];
        dst_row = ((id * H_kv + (bh % H_kv)) << page_shift) + (row & ((1 << page_shift) - 1));
    }
    const int64_t dst = dst_row * D + c * 8;
    const int64_t src = bh * D + c * 8;
    *reinterpret_cast<uint4*>(K + dst) = *reinterpret_cast<const uint4*>(k_new + src);
    *reinterpret_cast<uint4*>(V + dst) = *reinterpret_cast<const uint4*>(v_new + src);
}

__global__ void advance_kernel(int32_t* __restrict__ lens, int B)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) lens[b] += 1;
}

}  // namespace lckv
