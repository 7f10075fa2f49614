// Prompt encoding: token-parallel causal attention of one layer over a cache slot.
//
// Every prompt token i < len[b] attends rows j < i (condensed layers, diagonal masked) or j <= i
// (warmup layers) of the slot.  This is a dense contraction, so it runs on the tensor cores: one
// CTA owns 64 query rows of one (sequence, query head), four warps of 16 rows each; K and V tiles
// of 64 rows arrive by 2-D tiled TMA (128-byte swizzle, two stages); S = Q K^T and O += P V are
// bf16 m16n8k16 MMAs with fp32 accumulation and the usual running-max softmax in registers.
#pragma once
#include <cuda.h>

#include "lckv_attn_mma.cuh"

namespace lckv {

constexpr int kPfBM = 64;     // query rows per CTA
constexpr int kPfBN = 64;     // cache rows per tile
constexpr int kPfWarps = 4;
constexpr int kPfStages = 2;

template <int D>
constexpr int prefill_smem_bytes()
{
    return kPfStages * 2 * (kPfBN * D * 2) + 64 + 1024;  // K and V tiles, barriers, alignment slack
}

struct PrefillParams {
    const uint16_t* q;   // [B, n_max, H_q, D] bf16
    void* out;           // [B, n_max, H_q, D] bf16 or fp32
    const int32_t* lens; // [B] prompt lengths
    int32_t* status;
    int64_t T_cap;
    int32_t B, n_max, H_q, H_kv, mode, out_f32;
    float scale_log2;
    const int32_t* page_table;  // paged slots: [B_max][pt_stride] page ids, else null
    int32_t pt_stride, page_shift;
};

// First cache row (of the 2-D [rows, D] view of a slot) of the 64-row tile jt of (b, kv head).
__device__ __forceinline__ int64_t prefill_tile_row(const PrefillParams& p, int b, int kvh, int jt,
                                                    int tile_rows)
{
    const int r0 = jt * tile_rows;
    if (p.page_table) {   // a tile never straddles pages: the page size is a multiple of 64
        const int64_t id = __ldg(p.page_table + (size_t)b * p.pt_stride + (r0 >> p.page_shift));
        return ((id * p.H_kv + kvh) << p.page_shift) + (r0 & ((1 << p.page_shift) - 1));
    }
    return ((int64_t)b * p.H_kv + kvh) * p.T_cap + r0;
}

template <int D>
__global__ void __launch_bounds__(kPfWarps * 32)
prefill_attn_kernel(const PrefillParams p, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV)
{
    constexpr int KS = D / 16;           // k-steps of S = Q K^T
    constexpr int ND = D / 8;            // 8-column n-tiles of O
    constexpr int NBOX = D / 64;         // 64-column TMA boxes per tile
    constexpr int BOXB = kPfBN * 128;    // bytes of one box
    constexpr int TILEB = kPfBN * D * 2; // bytes of one K (or V) tile
    const uint32_t FULL = 0xffffffffu;

    const int b = blockIdx.z, h = blockIdx.y;
    const int mb = (int)gridDim.x - 1 - (int)blockIdx.x;  // long rows first
    const int nb = min(__ldg(p.lens + b), p.n_max);
    if (mb * kPfBM >= nb) return;
    const int g = p.H_q / p.H_kv;
    const int kvh = h / g;
    const int n_kv = mb + 1;             // tiles 0 .. mb reach the diagonal

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = smem0 + kPfStages * 2 * TILEB;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g4 = lane >> 2, c4 = lane & 3;
    if (tid == 0) {
        for (int s = 0; s < kPfStages; ++s) mbar_init(bars + 8 * s, 1);
        fence_mbar_init();
    }
    __syncthreads();

    auto issue = [&](int jt) {  // thread 0 only
        const int s = jt & 1;
        const uint32_t kb = smem0 + s * 2 * TILEB, vb = kb + TILEB;
        const int32_t row = (int32_t)prefill_tile_row(p, b, kvh, jt, kPfBN);
        mbar_expect_tx(bars + 8 * s, 2 * TILEB);
#pragma unroll
        for (int bx = 0; bx < NBOX; ++bx) {
            tma_load_2d(kb + bx * BOXB, &tmK, bx * 64, row, bars + 8 * s);
            tma_load_2d(vb + bx * BOXB, &tmV, bx * 64, row, bars + 8 * s);
        }
    };
    if (tid == 0) issue(0);

    // Q fragments of this warp's 16 rows (rows past the prompt read as zero)
    const int i0 = mb * kPfBM + warp * 16;
    const int ia = i0 + g4, ib = ia + 8;
    uint32_t qa[KS][4];
    {
        const uint16_t* qra = p.q + (((size_t)b * p.n_max + ia) * p.H_q + h) * D + 2 * c4;
        const uint16_t* qrb = p.q + (((size_t)b * p.n_max + ib) * p.H_q + h) * D + 2 * c4;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qa[ks][0] = ia < nb ? __ldg(reinterpret_cast<const uint32_t*>(qra + 16 * ks)) : 0u;
            qa[ks][1] = ib < nb ? __ldg(reinterpret_cast<const uint32_t*>(qrb + 16 * ks)) : 0u;
            qa[ks][2] = ia < nb ? __ldg(reinterpret_cast<const uint32_t*>(qra + 16 * ks + 8)) : 0u;
            qa[ks][3] = ib < nb ? __ldg(reinterpret_cast<const uint32_t*>(qrb + 16 * ks + 8)) : 0u;
        }
    }

    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o[ND][4];
#pragma unroll
    for (int nd = 0; nd < ND; ++nd)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[nd][e] = 0.f;

    bool ok = true;
    for (int jt = 0; jt < n_kv; ++jt) {
        const int s = jt & 1;
        if (tid == 0 && jt + 1 < n_kv) issue(jt + 1);  // its stage was released by the last sync
        const bool landed = mbar_wait_bounded(bars + 8 * s, (jt >> 1) & 1);
        if (!__syncthreads_and(landed)) { ok = false; break; }
        const uint32_t kb = smem0 + s * 2 * TILEB, vb = kb + TILEB;
        const int rows_valid = nb - jt * kPfBN;  // rows of this tile that belong to the prompt
        if (rows_valid < kPfBN) {
            // rows past the prompt came with the box: never visible, but 0 * NaN = NaN in the MMA
#pragma unroll
            for (int bx = 0; bx < NBOX; ++bx)
                for (int i = rows_valid * 128 + tid * 16; i < BOXB; i += kPfWarps * 32 * 16)
                    sts128(vb + bx * BOXB + i, make_uint4(0, 0, 0, 0));
            fence_proxy_async_smem();
            __syncthreads();
        }

        // ---- S = Q K^T -----------------------------------------------------------------------
        float sc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) sc[nt][e] = 0.f;
        {
            const int mi = lane >> 3;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const int chunk = 2 * ks + (mi & 1);
#pragma unroll
                for (int ntp = 0; ntp < 4; ++ntp) {
                    const int tok = (2 * ntp + (mi >> 1)) * 8 + (lane & 7);
                    const uint32_t addr = kb + (chunk >> 3) * BOXB + tok * 128 +
                                          (((chunk & 7) ^ (tok & 7)) << 4);
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4(addr, b0, b1, b2, b3);
                    mma_bf16_16816(sc[2 * ntp], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                    mma_bf16_16816(sc[2 * ntp + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b2, b3);
                }
            }
        }

        // ---- mask (only the diagonal tile needs it), running max, probabilities ----------------
        const bool diag = (jt == mb);
        float mt[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int col = jt * kPfBN + nt * 8 + 2 * c4 + (e & 1);
                const int row = (e >> 1) ? ib : ia;
                float v = sc[nt][e] * p.scale_log2;
                if (diag && !(col < row + p.mode)) v = -INFINITY;
                sc[nt][e] = v;
                mt[e >> 1] = fmaxf(mt[e >> 1], v);
            }
        float alpha[2], m_use[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mt[r] = fmaxf(mt[r], __shfl_xor_sync(FULL, mt[r], 1));
            mt[r] = fmaxf(mt[r], __shfl_xor_sync(FULL, mt[r], 2));
            const float m_new = fmaxf(m_run[r], mt[r]);
            m_use[r] = (m_new == -INFINITY) ? 0.f : m_new;  // a row that has seen nothing yet
            alpha[r] = ex2(m_run[r] - m_use[r]);
            m_run[r] = m_new;
            l_run[r] *= alpha[r];
        }
#pragma unroll
        for (int nd = 0; nd < ND; ++nd) {
            o[nd][0] *= alpha[0]; o[nd][1] *= alpha[0];
            o[nd][2] *= alpha[1]; o[nd][3] *= alpha[1];
        }
        uint32_t pa[4][4];  // P as the A operand: k-step j covers tile rows 16j .. 16j+15
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const uint32_t lo_pack = cvt_bf16x2(ex2(sc[nt][0] - m_use[0]), ex2(sc[nt][1] - m_use[0]));
            const uint32_t hi_pack = cvt_bf16x2(ex2(sc[nt][2] - m_use[1]), ex2(sc[nt][3] - m_use[1]));
            l_run[0] += bf16lo(lo_pack) + bf16hi(lo_pack);
            l_run[1] += bf16lo(hi_pack) + bf16hi(hi_pack);
            pa[nt >> 1][(nt & 1) * 2] = lo_pack;
            pa[nt >> 1][(nt & 1) * 2 + 1] = hi_pack;
        }

        // ---- O += P V --------------------------------------------------------------------------
        {
            const int mi = lane >> 3;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int tok = 16 * j + (mi & 1) * 8 + (lane & 7);
#pragma unroll
                for (int ndp = 0; ndp < ND / 2; ++ndp) {
                    const int chunk = 2 * ndp + (mi >> 1);
                    const uint32_t addr = vb + (chunk >> 3) * BOXB + tok * 128 +
                                          (((chunk & 7) ^ (tok & 7)) << 4);
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(addr, b0, b1, b2, b3);
                    mma_bf16_16816(o[2 * ndp], pa[j][0], pa[j][1], pa[j][2], pa[j][3], b0, b1);
                    mma_bf16_16816(o[2 * ndp + 1], pa[j][0], pa[j][1], pa[j][2], pa[j][3], b2, b3);
                }
            }
        }
        __syncthreads();  // everyone is done with this stage before it is refilled
    }

    if (!ok) {
        if (tid == 0) atomicExch(p.status, kStatusTimeout);
        for (int s = 0; s < kPfStages; ++s) {
            mbar_wait_bounded(bars + 8 * s, 0, 1u << 10);
            mbar_wait_bounded(bars + 8 * s, 1, 1u << 10);
        }
        return;
    }

    // ---- normalise and store ---------------------------------------------------------------------
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(FULL, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(FULL, l_run[r], 2);
    }
    const float inv0 = l_run[0] > 0.f ? 1.0f / l_run[0] : 0.f;  // nothing visible: zero dummy KV
    const float inv1 = l_run[1] > 0.f ? 1.0f / l_run[1] : 0.f;
    const size_t ra = (((size_t)b * p.n_max + ia) * p.H_q + h) * D + 2 * c4;
    const size_t rb = (((size_t)b * p.n_max + ib) * p.H_q + h) * D + 2 * c4;
#pragma unroll
    for (int nd = 0; nd < ND; ++nd) {
        if (p.out_f32) {
            float* ob = static_cast<float*>(p.out);
            if (ia < nb) *reinterpret_cast<float2*>(ob + ra + nd * 8) = make_float2(o[nd][0] * inv0, o[nd][1] * inv0);
            if (ib < nb) *reinterpret_cast<float2*>(ob + rb + nd * 8) = make_float2(o[nd][2] * inv1, o[nd][3] * inv1);
        } else {
            uint16_t* ob = static_cast<uint16_t*>(p.out);
            if (ia < nb) *reinterpret_cast<uint32_t*>(ob + ra + nd * 8) = cvt_bf16x2(o[nd][0] * inv0, o[nd][1] * inv0);
            if (ib < nb) *reinterpret_cast<uint32_t*>(ob + rb + nd * 8) = cvt_bf16x2(o[nd][2] * inv1, o[nd][3] * inv1);
        }
    }
}

// Rows [0, len[b]) of a slot <- the prompt's k, v given token-major [B, n_max, H_kv, D].
__global__ void prefill_write_kv_kernel(uint16_t* __restrict__ K, uint16_t* __restrict__ V,
                                        const uint16_t* __restrict__ k, const uint16_t* __restrict__ v,
                                        const int32_t* __restrict__ lens, int B, int n_max, int H_kv,
                                        int64_t T_cap, int D, const int32_t* __restrict__ page_table,
                                        int pt_stride, int page_shift)
{
    const int chunks = D / 8;
    const int64_t n = (int64_t)B * n_max * H_kv * chunks;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int c = (int)(i % chunks);
    const int hh = (int)((i / chunks) % H_kv);
    const int tok = (int)((i / ((int64_t)chunks * H_kv)) % n_max);
    const int b = (int)(i / ((int64_t)chunks * H_kv * n_max));
    if (tok >= lens[b] || tok >= T_cap) return;
    int64_t dst_row = (((int64_t)b * H_kv + hh) * T_cap) + tok;
    if (page_table) {
        const int64_t id = page_table[(int64_t)b * pt_stride + (tok >> page_shift)];
        dst_row = ((id * H_kv + hh) << page_shift) + (tok & ((1 << page_shift) - 1));
    }
    const int64_t dst = dst_row * D + c * 8;
    const int64_t src = (((int64_t)b * n_max + tok) * H_kv + hh) * (int64_t)D + c * 8;
    *reinterpret_cast<uint4*>(K + dst) = *reinterpret_cast<const uint4*>(k + src);
    *reinterpret_cast<uint4*>(V + dst) = *reinterpret_cast<const uint4*>(v + src);
}

}  // namespace lckv
