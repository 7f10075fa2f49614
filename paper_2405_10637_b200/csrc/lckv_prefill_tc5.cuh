// Prompt encoding on the 5th-generation tensor cores (tcgen05 + tensor memory).
//
// Same operation as prefill_attn_kernel (lckv_prefill.cuh): every prompt token i < len[b] attends
// cache rows j < i + mode of one slot.  One CTA owns 128 query rows of one (sequence, query head):
//
//   warp 0   producer: TMA loads of the Q tile (once) and of the 64-row K and V tiles
//   warp 1   one thread issues the MMAs:  S[128x64]  = Q K^T      (A, B from shared memory)
//                                         O[128xD]  += P V        (P from tensor memory, V MN-major)
//            accumulators live in tensor memory; completion is signalled by tcgen05.commit
//   warps 2-5  one thread per query row (= one tensor-memory lane): read the row of S, mask, running
//            max (thread-local, no shuffles), probabilities -> packed bf16 pairs back into tensor
//            memory (the A operand of the second MMA), row sum; rescale the O row in tensor memory
//            only when the maximum grew by more than 2^8 (the probabilities then stay <= 256);
//            epilogue.
//
// K and V tiles are double-buffered so that their load latency is hidden behind the previous
// tile.  Two CTAs fit on an SM (97 KB of shared memory and 256 of the 512 tensor-memory columns
// each at D = 128), so one CTA's softmax overlaps the other's MMAs.  Every wait is bounded.
#pragma once
#include <cuda.h>

#include "lckv_prefill.cuh"

namespace lckv {

constexpr int kT5BM = 128;   // query rows per CTA
constexpr int kT5BN = 64;    // cache rows per tile
constexpr int kT5Threads = 192;
constexpr uint32_t kT5WaitLimit = 1u << 16;

template <int D>
constexpr int tc5_smem_bytes()
{
    // Q [128 x D] + two stages of K [64 x D] and V [64 x D], bf16; barriers; alignment slack
    return kT5BM * D * 2 + 4 * kT5BN * D * 2 + 256 + 1024;
}

// ---- tcgen05 wrappers ----------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst),
                 "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tc5_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc5_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void tc5_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                        uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Same with the A operand in tensor memory (128 lanes = rows, K elements packed two per column).
__device__ __forceinline__ void tc5_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc,
                                           uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier receives one arrival once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void tc5_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive 32-bit columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
          "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
          "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
          "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
          "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
          "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
          "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),
          "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]),
          "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]),
          "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
          "r"(r[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor for a tile stored as rows of 128 bytes with the 128-byte swizzle
// (what a 64-column bf16 TMA box produces), base 1024-byte aligned.
//   K-major operand (rows = M or N, the 128 bytes run along K): groups of 8 rows are 1024 bytes
//     apart (SBO); the leading offset is not used.
//   MN-major operand (rows = K, the 128 bytes run along N): SBO = 1024 between groups of 8 K rows,
//     LBO = distance between consecutive 64-column blocks of N.
__device__ __forceinline__ uint64_t tc5_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);         // bits 0-13: start address / 16
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;    // bits 16-29
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;    // bits 32-45
    d |= (uint64_t)1 << 46;                               // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                               // 128-byte swizzle
    return d;
}

// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t tc5_idesc(int M, int N, int b_mn_major)
{
    return (1u << 4)                       // accumulator fp32
           | (1u << 7) | (1u << 10)        // A, B bf16
           | ((uint32_t)b_mn_major << 16)  // B major-ness (bit 15 = A: K-major)
           | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

template <int D>
__global__ void __launch_bounds__(kT5Threads)
prefill_tc5_kernel(const PrefillParams p, const __grid_constant__ CUtensorMap tmQ,
                   const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV)
{
    constexpr int NBOX = D / 64;                   // 64-column boxes per tile
    constexpr int QBOX = kT5BM * 128;              // bytes of one Q box
    constexpr int KBOX = kT5BN * 128;              // bytes of one K or V box
    constexpr int Q_BYTES = kT5BM * D * 2, KV_BYTES = kT5BN * D * 2;
    constexpr uint32_t TM_COLS = 256;   // 2 x S/P (64 columns each) + O (D fp32), power of two
    constexpr uint32_t IDESC_S = tc5_idesc(kT5BM, kT5BN, 0);
    constexpr uint32_t IDESC_O = tc5_idesc(kT5BM, D, 1);

    const int b = blockIdx.z, h = blockIdx.y;
    const int mb = (int)gridDim.x - 1 - (int)blockIdx.x;
    const int nb = min(__ldg(p.lens + b), p.n_max);
    if (mb * kT5BM >= nb) return;
    const int g = p.H_q / p.H_kv;
    const int kvh = h / g;
    const int i_max = min(mb * kT5BM + kT5BM - 1, nb - 1);
    const int c_last = i_max - 1 + p.mode;         // last cache row any query of this block sees
    const int n_kv = c_last < 0 ? 0 : c_last / kT5BN + 1;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem0, sK = sQ + Q_BYTES, sV = sK + 2 * KV_BYTES;   // K, V: two stages each
    const uint32_t bars = sV + 2 * KV_BYTES;
    // per-stage barriers are 8 bytes apart: bKf + 8 * stage etc.
    const uint32_t bQ = bars, bKf = bars + 8, bKe = bars + 24, bVf = bars + 40, bVe = bars + 56,
                   bSf = bars + 72, bPf = bars + 88, bOf = bars + 96, sTaddr = bars + 104;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (n_kv == 0) {
        // the block's only visible set is empty (first token under the diagonal mask): zeros
        for (int i = mb * kT5BM + (tid >> 4); i <= i_max; i += kT5Threads >> 4) {
            const size_t off = (((size_t)b * p.n_max + i) * p.H_q + h) * D;
            for (int c = (tid & 15); c < D * (p.out_f32 ? 4 : 2) / 16; c += 16)
                reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.out) + off * (p.out_f32 ? 4 : 2))[c] =
                    make_uint4(0, 0, 0, 0);
        }
        return;
    }

    if (tid == 0) {
        mbar_init(bQ, 1);
        for (int st = 0; st < 2; ++st) {
            mbar_init(bKf + 8 * st, 1); mbar_init(bKe + 8 * st, 1);
            mbar_init(bVf + 8 * st, 1); mbar_init(bVe + 8 * st, 1);
        }
        mbar_init(bSf, 1); mbar_init(bSf + 8, 1); mbar_init(bPf, 128); mbar_init(bOf, 1);
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(sTaddr, TM_COLS);
    tc5_fence_before();
    __syncthreads();
    tc5_fence_after();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(sTaddr));
    // Tensor memory: two score buffers of 64 columns (tile j uses buffer j & 1; the bf16 pairs of
    // P_j overwrite the first 32 columns of S_j once the row has been read), then O.
    const uint32_t tSP = tmem_base, tO = tmem_base + 2 * kT5BN;

    bool ok = true;
    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            mbar_expect_tx(bQ, Q_BYTES);
#pragma unroll
            for (int bx = 0; bx < NBOX; ++bx)
                tma_load_2d(sQ + bx * QBOX, &tmQ, h * D + bx * 64, b * p.n_max + mb * kT5BM, bQ);
            for (int j = 0; j < n_kv && ok; ++j) {
                const int st = j & 1;                    // stage; its k-th use has parity k & 1
                const uint32_t par_prev = ((j >> 1) - 1) & 1;
                if (j >= 2) ok = mbar_wait_bounded(bKe + 8 * st, par_prev, kT5WaitLimit);
                if (!ok) break;
                const int32_t row = (int32_t)prefill_tile_row(p, b, kvh, j, kT5BN);
                mbar_expect_tx(bKf + 8 * st, KV_BYTES);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx)
                    tma_load_2d(sK + st * KV_BYTES + bx * KBOX, &tmK, bx * 64, row, bKf + 8 * st);
                if (j >= 2) ok = mbar_wait_bounded(bVe + 8 * st, par_prev, kT5WaitLimit);
                if (!ok) break;
                mbar_expect_tx(bVf + 8 * st, KV_BYTES);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx)
                    tma_load_2d(sV + st * KV_BYTES + bx * KBOX, &tmV, bx * 64, row, bVf + 8 * st);
            }
            if (!ok) atomicExch(p.status, kStatusTimeout);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            ok = mbar_wait_bounded(bQ, 0, kT5WaitLimit);
            // S_t = Q K_t^T into score buffer t & 1
            auto issue_s = [&](int t) {
                const uint32_t kb = sK + (t & 1) * KV_BYTES;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint64_t ad = tc5_desc(sQ + (ks >> 2) * QBOX + (ks & 3) * 32, 16, 1024);
                    const uint64_t bd = tc5_desc(kb + (ks >> 2) * KBOX + (ks & 3) * 32, 16, 1024);
                    tc5_mma(tSP + (t & 1) * kT5BN, ad, bd, IDESC_S, ks > 0);
                }
                tc5_commit(bSf + 8 * (t & 1));   // S_t ready for the softmax threads
                tc5_commit(bKe + 8 * (t & 1));   // K stage may be refilled
            };
            // O += P_t V_t (P in tensor memory, buffer t & 1; V tile in stage t & 1)
            auto issue_pv = [&](int t) {
                const uint32_t vb = sV + (t & 1) * KV_BYTES;
#pragma unroll
                for (int ks = 0; ks < kT5BN / 16; ++ks) {
                    const uint64_t bd = tc5_desc(vb + ks * 16 * 128, KBOX, 1024);
                    tc5_mma_ts(tO, tSP + (t & 1) * kT5BN + ks * 8, bd, IDESC_O, (t > 0 || ks > 0));
                }
                tc5_commit(bOf);                 // O free for rescaling, score buffer t & 1 reusable
                tc5_commit(bVe + 8 * (t & 1));   // V stage may be refilled
            };
            if (ok) ok = mbar_wait_bounded(bKf, 0, kT5WaitLimit);
            if (ok) { tc5_fence_after(); issue_s(0); }
            for (int j = 0; j < n_kv && ok; ++j) {
                if (j + 1 < n_kv) {
                    // scores of the next tile, one tile ahead of the softmax: needs K_{j+1} and the
                    // buffer (j+1) & 1, whose last user was P_{j-1} V_{j-1}
                    ok = mbar_wait_bounded(bKf + 8 * ((j + 1) & 1), ((j + 1) >> 1) & 1, kT5WaitLimit);
                    if (ok && j >= 1) ok = mbar_wait_bounded(bOf, (j - 1) & 1, kT5WaitLimit);
                    if (!ok) break;
                    tc5_fence_after();
                    issue_s(j + 1);
                }
                ok = mbar_wait_bounded(bPf, j & 1, kT5WaitLimit) &&
                     mbar_wait_bounded(bVf + 8 * (j & 1), (j >> 1) & 1, kT5WaitLimit);
                if (!ok) break;
                tc5_fence_after();
                issue_pv(j);
            }
            if (!ok) atomicExch(p.status, kStatusTimeout);
        }
    } else {
        // ------------------------------------------------------------------ softmax: one row per thread
        const int q4 = warp & 3;                       // tensor-memory lane quarter of this warp
        const int r = q4 * 32 + lane;                  // row within the block
        const int i = mb * kT5BM + r;                  // prompt position of the row
        const uint32_t lane_sel = (uint32_t)(q4 * 32) << 16;
        float m_used = -INFINITY, l_run = 0.f;     // m_used in raw (unscaled) score units
        const float inv_scale = 1.0f / p.scale_log2;
        for (int j = 0; j < n_kv && ok; ++j) {
            ok = mbar_wait_bounded(bSf + 8 * (j & 1), (j >> 1) & 1, kT5WaitLimit);
            if (!ok) break;
            tc5_fence_after();
            uint32_t s0[32], s1[32];
            const uint32_t tbuf = tSP + (j & 1) * kT5BN + lane_sel;
            tmem_ld32_nowait(tbuf, s0);
            tmem_ld32_nowait(tbuf + 32, s1);
            tmem_ld_wait();
            // Raw scores stay unscaled: the (positive) scale is folded into the exponent's FMA.
            const bool need_mask = (j * kT5BN + kT5BN > mb * kT5BM + p.mode);  // tile reaches the diagonal
            float mt = -INFINITY;
            if (need_mask) {
                const int lim = i + p.mode - j * kT5BN;   // columns c < lim are visible
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    if (c >= lim) s0[c] = 0xff800000u;       // -inf
                    if (c + 32 >= lim) s1[c] = 0xff800000u;
                }
            }
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
                mt = fmaxf(mt, fmaxf(__uint_as_float(s0[c]), __uint_as_float(s0[c + 1])));
                mt = fmaxf(mt, fmaxf(__uint_as_float(s1[c]), __uint_as_float(s1[c + 1])));
            }
            // Keep the reference maximum unless the new one exceeds it by more than 2^8 (in the
            // exponent's base-2 units): probabilities then stay <= 256.
            float alpha = 1.f;
            const bool grow = (mt > m_used + 8.f * inv_scale) || (m_used == -INFINITY && mt > -INFINITY);
            if (grow) {
                alpha = ex2((m_used - mt) * p.scale_log2);   // 0 when nothing was seen before
                m_used = mt;
                l_run *= alpha;
            }
            const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used * p.scale_log2;
            uint32_t pk[32];
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const float p0 = ex2(fmaf(__uint_as_float(s0[2 * c]), p.scale_log2, neg_m));
                const float p1 = ex2(fmaf(__uint_as_float(s0[2 * c + 1]), p.scale_log2, neg_m));
                const float p2 = ex2(fmaf(__uint_as_float(s1[2 * c]), p.scale_log2, neg_m));
                const float p3 = ex2(fmaf(__uint_as_float(s1[2 * c + 1]), p.scale_log2, neg_m));
                pk[c] = cvt_bf16x2(p0, p1);
                pk[c + 16] = cvt_bf16x2(p2, p3);
                l_run += (p0 + p1) + (p2 + p3);
            }
            // P and O are still in use by the previous tile's P V until O_full fires
            if (j > 0) {
                ok = mbar_wait_bounded(bOf, (j - 1) & 1, kT5WaitLimit);
                if (!ok) break;
                tc5_fence_after();
                if (__any_sync(0xffffffffu, grow)) {
#pragma unroll 1
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        uint32_t ov[32];
                        tmem_ld32(tO + lane_sel + c0, ov);
#pragma unroll
                        for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
                        tmem_st32(tO + lane_sel + c0, ov);
                    }
                }
            }
            // row r of P: 64 bf16 as 32 packed pairs = 32 tensor-memory columns of this lane
            tmem_st32(tbuf, pk);
            if (j * kT5BN + kT5BN > nb) {
                // rows of V past the prompt came with the box: weight 0, but 0 * NaN = NaN
                ok = mbar_wait_bounded(bVf + 8 * (j & 1), (j >> 1) & 1, kT5WaitLimit);
                if (!ok) break;
                const int first = nb - j * kT5BN;
                const int t128 = tid - 64;
                const uint32_t vb = sV + (j & 1) * KV_BYTES;
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx)
                    for (int x = first * 128 + t128 * 16; x < KBOX; x += 128 * 16)
                        sts128(vb + bx * KBOX + x, make_uint4(0, 0, 0, 0));
                fence_proxy_async_smem();   // generic writes -> visible to the MMA's reads
            }
            tc5_fence_before();
            mbar_arrive(bPf);
        }
        if (ok) ok = mbar_wait_bounded(bOf, (n_kv - 1) & 1, kT5WaitLimit);
        if (ok) {
            tc5_fence_after();
            const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
            // tcgen05.ld is warp-collective: every lane loads, only rows of the prompt store
            const size_t off = (((size_t)b * p.n_max + min(i, p.n_max - 1)) * p.H_q + h) * D;
#pragma unroll 1
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t ov[32];
                tmem_ld32(tO + lane_sel + c0, ov);
                if (i < nb) {
                    if (p.out_f32) {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.out) + off + c0);
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            dst[c] = make_float4(__uint_as_float(ov[4 * c]) * inv, __uint_as_float(ov[4 * c + 1]) * inv,
                                                 __uint_as_float(ov[4 * c + 2]) * inv, __uint_as_float(ov[4 * c + 3]) * inv);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + off + c0);
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            dst[c] = make_uint4(
                                cvt_bf16x2(__uint_as_float(ov[8 * c]) * inv, __uint_as_float(ov[8 * c + 1]) * inv),
                                cvt_bf16x2(__uint_as_float(ov[8 * c + 2]) * inv, __uint_as_float(ov[8 * c + 3]) * inv),
                                cvt_bf16x2(__uint_as_float(ov[8 * c + 4]) * inv, __uint_as_float(ov[8 * c + 5]) * inv),
                                cvt_bf16x2(__uint_as_float(ov[8 * c + 6]) * inv, __uint_as_float(ov[8 * c + 7]) * inv));
                    }
                }
            }
        } else if (lane == 0) {
            atomicExch(p.status, kStatusTimeout);
        }
    }

    tc5_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, TM_COLS);
}

}  // namespace lckv
