// Decode attention, tensor-core kernel for grouped-query attention: the 8 query heads that share a
// kv head form the N = 8 side of a dense bf16 m16n8k16 MMA tile.  Groups of 2 ... 7 use the same
// tile with zero queries in the unused columns (K and V are still read once per group, which is
// what matters: the work is streaming them); larger groups are split into pairs of 8.
//
//   S^T [tokens x 8] = K [tokens x d] . Q^T [d x 8]        (tokens are the M dimension)
//   O^T [d x 8]      = V^T [d x tokens] . P^T [tokens x 8]
//
// Work decomposition, per-warp copy ring, running-max softmax and the ticketed merge of split
// pairs are those of the FP32-ALU kernel (lckv_attn_alu.cuh); a pair here is (sequence, group of up to 8
// query heads).  Differences: tiles arrive through 2-D tiled TMA with the 128-byte swizzle so that
// ldmatrix reads them without bank conflicts; the probabilities are rounded to bf16 for the second
// MMA (their sum is taken over the rounded values, so the weights stay normalised); a TMA box is
// always whole, so rows past the visible count are fetched, masked in the scores and zeroed in V.
#pragma once
#include <cuda.h>

#include "lckv_attn_alu.cuh"

namespace lckv {

#ifndef LCKV_MMA_WARPS
#define LCKV_MMA_WARPS 8
#endif
#ifndef LCKV_MMA_SLOTS
#define LCKV_MMA_SLOTS 2
#endif
#ifndef LCKV_MMA_CTAS
#define LCKV_MMA_CTAS 1
#endif
constexpr int kMmaWarps = LCKV_MMA_WARPS;   // workers per CTA
constexpr int kMmaCtas = LCKV_MMA_CTAS;     // CTAs per SM
constexpr int kMmaSlots = LCKV_MMA_SLOTS;
#ifndef LCKV_MMA_SLOT_BYTES
#define LCKV_MMA_SLOT_BYTES 8192
#endif
constexpr int kMmaSlotBytes = LCKV_MMA_SLOT_BYTES;
constexpr int kMmaSmemBytes = kMmaWarps * kMmaSlots * (kMmaSlotBytes + 8) + 1024;  // + alignment slack
constexpr int kMmaTreeMin = 24;   // pairs split over more workers than this are merged in two levels
constexpr int kMmaChunk = 16;     // contributors per first-level chunk

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                            uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1,
                                                  uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// {lo, hi} -> packed bf16x2 (round to nearest even), lo in the low half.
__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// Position in a launch's tile sequence, with everything a copy needs kept incrementally (no
// division or 64-bit multiply per tile).
struct RowCursor {
    int32_t b, h;      // sequence; pair within the sequence
    uint32_t t, nt;    // tile within the pair; tiles per pair of sequence b
    int32_t nv;        // visible rows of sequence b
    uint32_t pre0;     // tiles (per pair index) of the sequences before b
    int32_t kvh, sub;  // kv head the pair reads; index of the pair among the pairs of that kv head
    int64_t row;       // cache row (of the [B*H_kv*T_cap, D] view) where the tile starts
};

__device__ __forceinline__ void rcursor_load(RowCursor& c, const AttnParams& p)
{
    c.pre0 = __ldg(p.pre + c.b);
    c.nt = __ldg(p.pre + c.b + 1) - c.pre0;
    c.nv = visible_rows(__ldg(p.lens + c.b), p.mode, p.T_cap);
}

// After b, h, t are set: derive the kv head and the tile's first row.  per_kv = pairs per kv head.
__device__ __forceinline__ void rcursor_seek(RowCursor& c, const AttnParams& p, int per_kv, int R)
{
    c.kvh = c.h / per_kv;
    c.sub = c.h - c.kvh * per_kv;
    c.row = ((int64_t)c.b * p.H_kv + c.kvh) * p.T_cap + (int64_t)c.t * R;
}

// Next tile in (b, pair, tile) order, skipping sequences without tiles.  Safe past the end.
__device__ __forceinline__ void rcursor_next(RowCursor& c, const AttnParams& p, int H, int per_kv,
                                            int R)
{
    if (++c.t < c.nt) { c.row += R; return; }
    c.t = 0;
    if (++c.h < H) {
        if (++c.sub == per_kv) { c.sub = 0; ++c.kvh; }
    } else {
        c.h = 0; c.sub = 0; c.kvh = 0;
        do {
            if (++c.b >= p.B) { c.b = p.B; c.nt = 0; c.nv = 0; return; }
            rcursor_load(c, p);
        } while (c.nt == 0);
    }
    c.row = ((int64_t)c.b * p.H_kv + c.kvh) * p.T_cap;
}

struct MmaParams {
    AttnParams a;     // H_q here = pairs per sequence (groups of up to 8 query heads); see the launcher
    int32_t n_q_heads;  // real H_q, for addressing q / out / lse
    int32_t groups_per_kv;  // pairs that share one kv head
    int32_t heads_per_pair; // query heads of a pair: 8, or the whole group when it is smaller (the
                            // other columns of the N = 8 tile then carry zero queries)
};

template <int D, bool PAGED = false>
__global__ void __launch_bounds__(kMmaWarps * 32, kMmaCtas)
attn_mma_kernel(const MmaParams mp, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV)
{
    constexpr int R = kMmaSlotBytes / (D * 2);  // tokens per tile: 64 (D=64), 32 (D=128)
    constexpr int RB = R / 16;                  // 16-token row blocks per tile
    constexpr int KS = D / 16;                  // k-steps of the score MMA
    constexpr int MT = D / 16;                  // 16-dim m-tiles of the output MMA
    constexpr int NBOX = D / 64;                // 128-byte-wide TMA boxes per tile
    constexpr int BOX_BYTES = R * 128;
    constexpr int NS = kMmaSlots;
    constexpr int REC = D * 8 + 16;             // floats per partial record
    const AttnParams& p = mp.a;

    extern __shared__ uint8_t smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int w = blockIdx.x * kMmaWarps + warp;
    const int H = p.H_q;  // pairs per sequence
    const uint32_t FULL = 0xffffffffu;
    const int g4 = lane >> 2, c4 = lane & 3;
    const int HP = mp.heads_per_pair;

    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms are 1024 bytes
    const uint32_t ring = smem0 + warp * (NS * kMmaSlotBytes);
    const uint32_t bars = smem0 + kMmaWarps * NS * kMmaSlotBytes + warp * (NS * 8);
    if (lane == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(bars + 8 * s, 1);
        fence_mbar_init();
    }
    __syncwarp();

    if (!p.early_kv) pdl_wait_then_release();

    // (a launch may use fewer workers than the grid holds: the others have nothing to do)
    const bool in_range = w < p.n_workers;
    WorkerStart ws = {0, 0, 0u, 0u, 0, 0u, 0u, 0u};
    if (in_range) ws = load_worker_start(p.start + w);
    const uint64_t total = (uint64_t)__ldg(p.pre + p.B) * (uint64_t)H;   // (needed from the first cut pair on)
    const uint64_t n_eff = total < (uint64_t)p.n_workers ? total : (uint64_t)p.n_workers;
    const uint32_t n_tiles = ws.n_tiles;
    const bool has_work = n_tiles != 0;
    RowCursor cc;
    cc.b = ws.b; cc.h = ws.h; cc.t = ws.t; cc.nt = ws.nt; cc.nv = ws.nv; cc.pre0 = ws.pre0;
    cc.kvh = 0; cc.sub = 0; cc.row = 0;
    if (has_work) rcursor_seek(cc, p, mp.groups_per_kv, R);
    const uint32_t n_items = 2 * n_tiles;
    RowCursor ci = cc;

    const uint64_t l2pol = make_l2_policy(p.l2_keep);
    uint32_t issued = 0, islot = 0;
    PageWalker walker;
    auto issue = [&]() {
        int64_t row;
        if constexpr (PAGED) row = walker.row(p, ci.b, ci.kvh, (int)ci.t * R);
        else row = ci.row;
        if (lane == 0) {
            const void* tm = (issued & 1) ? (const void*)&tmV : (const void*)&tmK;
            mbar_expect_tx(bars + 8 * islot, kMmaSlotBytes);
#pragma unroll
            for (int bx = 0; bx < NBOX; ++bx)
                tma_load_2d_hint(ring + islot * kMmaSlotBytes + bx * BOX_BYTES, tm, bx * 64,
                                 (int32_t)row, bars + 8 * islot, l2pol);
        }
        if (issued & 1) rcursor_next(ci, p, H, mp.groups_per_kv, R);
        ++issued;
        islot = (islot + 1 == NS) ? 0 : islot + 1;
    };
    {
        const uint32_t pro = n_items < (uint32_t)NS ? n_items : (uint32_t)NS;
        while (issued < pro) issue();
    }
    if (p.early_kv) pdl_wait_then_release();

    // Sequences that see nothing: zero rows (zero dummy KV), lse 0.
    for (int b = in_range ? w : p.B; b < p.B; b += p.n_workers) {
        if (visible_rows(__ldg(p.lens + b), p.mode, p.T_cap) == 0) {
            const int esz = p.out_f32 ? 4 : 2;
            const int n16 = mp.n_q_heads * D * esz / 16;
            uint4* o16 = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.out) +
                                                  (size_t)b * mp.n_q_heads * D * esz);
            for (int i = lane; i < n16; i += 32) o16[i] = make_uint4(0, 0, 0, 0);
            if (p.lse)
                for (int i = lane; i < mp.n_q_heads; i += 32)
                    p.lse[(size_t)b * mp.n_q_heads + i] = 0.f;
        }
    }

    if (!has_work) return;

    uint32_t cslot = 0, cphase = 0;
    bool ok = true;

    // Q^T fragments of the pair's 8 query heads: lane holds query g4, dims 2*c4 (+1) (+8) per k-step.
    uint32_t qb[KS][2], qn[KS][2];
    auto load_q = [&](const RowCursor& c, uint32_t (&dst)[KS][2]) {
        const uint16_t* qp = p.q + ((size_t)c.b * mp.n_q_heads + (size_t)c.h * HP + g4) * D + 2 * c4;
        const bool real = g4 < HP;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            dst[ks][0] = real ? __ldg(reinterpret_cast<const uint32_t*>(qp + ks * 16)) : 0u;
            dst[ks][1] = real ? __ldg(reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8)) : 0u;
        }
    };
    load_q(cc, qb);
    uint32_t seg_t0 = cc.t;
    // running state for this lane's two queries (2*c4, 2*c4+1)
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[mt][i] = 0.f;

    // Tickets posted for the (at most two) pairs this worker shares with others: the pair its range
    // starts in the middle of (record 0) and the pair it ends in the middle of (record 1).  A ticket is
    // posted when the worker's part is done and looked at only after its last tile.
    struct Pending { int32_t ticket, n, first_odd, b, h; uint32_t c_first; bool armed; };
    Pending pend0 = {0, 0, 0, 0, 0, 0u, false}, pend1 = pend0;
    // Which workers share a pair: worked out when the worker enters a pair that its range cuts (at
    // most its first and its last), so that the divisions are off the path that ends the kernel.
    struct Split { uint32_t c_first; int32_t n_parts, first_odd; };
    auto split_of = [&](const RowCursor& c) {
        const uint64_t gs = (uint64_t)c.pre0 * (uint64_t)H + (uint64_t)c.h * c.nt;  // the pair's first global tile
        const uint64_t ge = gs + c.nt;
        Split sp;
        sp.c_first = (uint32_t)(((gs + 1) * n_eff - 1) / total);
        const uint32_t c_last = (uint32_t)((ge * n_eff - 1) / total);
        const uint64_t lo_first = (uint64_t)sp.c_first * total / n_eff;
        sp.first_odd = (gs != lo_first) ? 1 : 0;  // which record of c_first belongs to this pair
        sp.n_parts = (int32_t)(c_last - sp.c_first) + 1;
        return sp;
    };
    Split cur = {0u, 1, 0}, nxt = cur;
    if (cc.t != 0 || n_tiles < cc.nt) cur = split_of(cc);   // the first pair is cut by this range
    bool first_seg = true;                                  // still in the segment that starts at lo
    float l_tot[2] = {0.f, 0.f}, m_fin[2] = {0.f, 0.f};   // with o[][]: the result being stored or merged

    // o / l_tot, lse from (m_fin, l_tot) -> the output rows of pair (b, h)
    auto write_rows = [&](int b, int h) {
        const float inv0 = 1.0f / l_tot[0], inv1 = 1.0f / l_tot[1];
        const size_t row0 = (size_t)b * mp.n_q_heads + (size_t)h * HP;  // first q head
        const bool col0 = 2 * c4 < HP, col1 = 2 * c4 + 1 < HP;
        if (p.out_f32) {
            float* ob = static_cast<float*>(p.out);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const int d0 = mt * 16 + g4;
                if (col0) {
                    ob[(row0 + 2 * c4) * D + d0] = o[mt][0] * inv0;
                    ob[(row0 + 2 * c4) * D + d0 + 8] = o[mt][2] * inv0;
                }
                if (col1) {
                    ob[(row0 + 2 * c4 + 1) * D + d0] = o[mt][1] * inv1;
                    ob[(row0 + 2 * c4 + 1) * D + d0 + 8] = o[mt][3] * inv1;
                }
            }
        } else {
            // transpose the [dims x queries] fragments so a lane holds two adjacent dims of
            // one query: 4-byte stores, one query row per 8 lanes
            uint16_t* ob = static_cast<uint16_t*>(p.out) + (row0 + g4) * D + 2 * c4;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const uint32_t t0 = movmatrix_trans(cvt_bf16x2(o[mt][0] * inv0, o[mt][1] * inv1));
                const uint32_t t1 = movmatrix_trans(cvt_bf16x2(o[mt][2] * inv0, o[mt][3] * inv1));
                if (g4 < HP) {
                    *reinterpret_cast<uint32_t*>(ob + mt * 16) = t0;
                    *reinterpret_cast<uint32_t*>(ob + mt * 16 + 8) = t1;
                }
            }
        }
        if (p.lse && g4 == 0) {
            if (col0) p.lse[row0 + 2 * c4] = (m_fin[0] + lg2(l_tot[0])) * 0.6931471805599453f;
            if (col1) p.lse[row0 + 2 * c4 + 1] = (m_fin[1] + lg2(l_tot[1])) * 0.6931471805599453f;
        }
    };
    // (o, m_fin, l_tot) -> a partial record; accumulators in fragment order: fully coalesced
    auto store_record = [&](float* rec) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
            reinterpret_cast<float4*>(rec)[mt * 32 + lane] = make_float4(o[mt][0], o[mt][1], o[mt][2], o[mt][3]);
        if (g4 == 0) {
            rec[D * 8 + 2 * c4] = m_fin[0];     rec[D * 8 + 2 * c4 + 1] = m_fin[1];
            rec[D * 8 + 8 + 2 * c4] = l_tot[0]; rec[D * 8 + 8 + 2 * c4 + 1] = l_tot[1];
        }
    };
    // Merge of n records in a fixed order, in one pass with running maxima: record i is the one of
    // worker first_w + i * step (its second record if i == 0 and first_slot is set).  Record
    // addresses do not depend on loaded data, so the unrolled loop keeps several L2 round trips in
    // flight.  Leaves the merged (unnormalised) values in o, l_tot, m_fin.
    auto merge_records = [&](int n, uint32_t first_w, int step, int first_slot) {
        const float* rec0 = p.partials + (size_t)(2 * first_w) * REC;
        const size_t rstride = (size_t)(2 * step) * REC;
        float M[2] = {-INFINITY, -INFINITY}, Ls[2] = {0.f, 0.f};
        float acc[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
#pragma unroll 2
        for (int i = 0; i < n; ++i) {
            const float* r = rec0 + (size_t)i * rstride + (i == 0 ? (size_t)first_slot * REC : 0);
            const float2 mm = __ldcg(reinterpret_cast<const float2*>(r + D * 8) + c4);
            const float2 ll = __ldcg(reinterpret_cast<const float2*>(r + D * 8 + 8) + c4);
            float4 x[MT];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) x[mt] = __ldcg(reinterpret_cast<const float4*>(r) + mt * 32 + lane);
            const float M0 = fmaxf(M[0], mm.x), M1 = fmaxf(M[1], mm.y);
            const float a0 = ex2(M[0] - M0), a1 = ex2(M[1] - M1);      // ex2(-inf) = 0 for the first record
            const float w0 = ex2(mm.x - M0), w1 = ex2(mm.y - M1);
            M[0] = M0; M[1] = M1;
            Ls[0] = fmaf(Ls[0], a0, ll.x * w0);
            Ls[1] = fmaf(Ls[1], a1, ll.y * w1);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                acc[mt][0] = fmaf(acc[mt][0], a0, x[mt].x * w0);
                acc[mt][1] = fmaf(acc[mt][1], a1, x[mt].y * w1);
                acc[mt][2] = fmaf(acc[mt][2], a0, x[mt].z * w0);
                acc[mt][3] = fmaf(acc[mt][3], a1, x[mt].w * w1);
            }
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) o[mt][i] = acc[mt][i];
        l_tot[0] = Ls[0]; l_tot[1] = Ls[1];
        m_fin[0] = M[0]; m_fin[1] = M[1];
    };

    for (uint32_t tile = 0; tile < n_tiles; ++tile) {
        const int rows = min(R, cc.nv - (int)cc.t * R);
        const bool pair_end = (cc.t + 1 == cc.nt);
        const bool last = (tile + 1 == n_tiles);
        // the next pair's queries are fetched while this pair's last tile is worked on
        RowCursor cn = cc;
        if (pair_end && !last) {
            rcursor_next(cn, p, H, mp.groups_per_kv, R);
            if (n_tiles - (tile + 1) < cn.nt) nxt = split_of(cn);   // the range ends inside the next pair
            load_q(cn, qn);
        }

        // ---- K tile: S^T = K . Q^T ----------------------------------------------------------
        if (!mbar_wait_bounded(bars + 8 * cslot, cphase, p.wait_limit)) { ok = false; break; }
        float s[RB][4];
        {
            const uint32_t slot = ring + cslot * kMmaSlotBytes;
#pragma unroll
            for (int rb = 0; rb < RB; ++rb) {
#pragma unroll
                for (int i = 0; i < 4; ++i) s[rb][i] = 0.f;
                const int r = rb * 16 + (lane & 15);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int cg = 2 * ks + (lane >> 4);  // 16-byte chunk of the d-row
                    const uint32_t addr = slot + (cg >> 3) * BOX_BYTES + r * 128 +
                                          (((cg & 7) ^ (r & 7)) << 4);
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4(addr, a0, a1, a2, a3);
                    mma_bf16_16816(s[rb], a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
                }
            }
        }
        __syncwarp();
        if (issued < n_items) issue();
        cslot = (cslot + 1 == NS) ? 0 : cslot + 1;
        if (cslot == 0) cphase ^= 1;

        // scale to base-2 logits, mask rows past the visible count
        float mt_[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) {
            const int t0 = rb * 16 + g4, t1 = t0 + 8;
            s[rb][0] = (t0 < rows) ? s[rb][0] * p.scale_log2 : -INFINITY;
            s[rb][1] = (t0 < rows) ? s[rb][1] * p.scale_log2 : -INFINITY;
            s[rb][2] = (t1 < rows) ? s[rb][2] * p.scale_log2 : -INFINITY;
            s[rb][3] = (t1 < rows) ? s[rb][3] * p.scale_log2 : -INFINITY;
            mt_[0] = fmaxf(mt_[0], fmaxf(s[rb][0], s[rb][2]));
            mt_[1] = fmaxf(mt_[1], fmaxf(s[rb][1], s[rb][3]));
        }
#pragma unroll
        for (int off = 4; off <= 16; off <<= 1) {
            mt_[0] = fmaxf(mt_[0], __shfl_xor_sync(FULL, mt_[0], off));
            mt_[1] = fmaxf(mt_[1], __shfl_xor_sync(FULL, mt_[1], off));
        }
        float alpha[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float m_new = fmaxf(m_run[j], mt_[j]);
            alpha[j] = ex2(m_run[j] - m_new);
            m_run[j] = m_new;
            l_run[j] *= alpha[j];
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            o[mt][0] *= alpha[0]; o[mt][1] *= alpha[1];
            o[mt][2] *= alpha[0]; o[mt][3] *= alpha[1];
        }
        // probabilities -> bf16 pairs -> transposed into the B operand of the second MMA
        uint32_t pb[RB][2];
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) {
            const uint32_t lo_pack = cvt_bf16x2(ex2(s[rb][0] - m_run[0]), ex2(s[rb][1] - m_run[1]));
            const uint32_t hi_pack = cvt_bf16x2(ex2(s[rb][2] - m_run[0]), ex2(s[rb][3] - m_run[1]));
            l_run[0] += bf16lo(lo_pack) + bf16lo(hi_pack);
            l_run[1] += bf16hi(lo_pack) + bf16hi(hi_pack);
            pb[rb][0] = movmatrix_trans(lo_pack);
            pb[rb][1] = movmatrix_trans(hi_pack);
        }

        // ---- V tile: O^T += V^T . P^T -------------------------------------------------------
        if (!mbar_wait_bounded(bars + 8 * cslot, cphase, p.wait_limit)) { ok = false; break; }
        {
            const uint32_t slot = ring + cslot * kMmaSlotBytes;
            if (rows < R) {
                // rows past the visible count came along with the box: weight 0, but 0 * NaN = NaN
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx)
                    for (int i = rows * 128 + lane * 16; i < BOX_BYTES; i += 32 * 16)
                        sts128(slot + bx * BOX_BYTES + i, make_uint4(0, 0, 0, 0));
                fence_proxy_async_smem();
                __syncwarp();
            }
#pragma unroll
            for (int rb = 0; rb < RB; ++rb) {
                const int r = rb * 16 + (lane & 7) + ((lane >> 4) & 1) * 8;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const int cg = 2 * mt + ((lane >> 3) & 1);
                    const uint32_t addr = slot + (cg >> 3) * BOX_BYTES + r * 128 +
                                          (((cg & 7) ^ (r & 7)) << 4);
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4_trans(addr, a0, a1, a2, a3);
                    mma_bf16_16816(o[mt], a0, a1, a2, a3, pb[rb][0], pb[rb][1]);
                }
            }
        }
        __syncwarp();
        if (issued < n_items) issue();
        cslot = (cslot + 1 == NS) ? 0 : cslot + 1;
        if (cslot == 0) cphase ^= 1;

        // ---- end of this worker's part of the pair? -----------------------------------------
        if (pair_end || last) {
            l_tot[0] = l_run[0]; l_tot[1] = l_run[1];
#pragma unroll
            for (int off = 4; off <= 16; off <<= 1) {
                l_tot[0] += __shfl_xor_sync(FULL, l_tot[0], off);
                l_tot[1] += __shfl_xor_sync(FULL, l_tot[1], off);
            }
            m_fin[0] = m_run[0]; m_fin[1] = m_run[1];

            const bool complete = pair_end && seg_t0 == 0;
            if (complete) {
                write_rows(cc.b, cc.h);
            } else {
                const uint32_t c_first = cur.c_first;
                const int first_odd = cur.first_odd, n_parts = cur.n_parts;
                const bool at_lo = first_seg;
                store_record(p.partials + (size_t)(2 * w + (at_lo ? 0 : 1)) * REC);
                // Few parts: the contributor that arrives last merges them all.  Many parts (few
                // pairs, long sequences): two levels - the contributors of a pair form chunks of
                // kMmaChunk consecutive workers; the last arriver of a chunk merges the chunk's records
                // into the record of the chunk's first worker, and the last chunk to finish merges
                // the chunk records.  Same fixed order either way.
                const bool two_level = n_parts > kMmaTreeMin && p.counters2 != nullptr;
                if (!two_level) {
                    // Post the ticket now (the release and the atomic's flight overlap with the copies
                    // of the next tiles, already on their way); the answer is looked at after the last
                    // tile.  Each ticket goes straight into its own variable: nothing may consume the
                    // atomic's result here, or the warp would wait for the round trip after all.
                    __syncwarp();   // the record's stores (all lanes) are ordered before lane 0's release
                    if (at_lo) {
                        if (lane == 0) pend0.ticket = atom_add_acq_rel_gpu(p.counters + c_first, 1);
                        pend0.n = n_parts; pend0.first_odd = first_odd; pend0.b = cc.b; pend0.h = cc.h;
                        pend0.c_first = c_first; pend0.armed = true;
                    } else {
                        if (lane == 0) pend1.ticket = atom_add_acq_rel_gpu(p.counters + c_first, 1);
                        pend1.n = n_parts; pend1.first_odd = first_odd; pend1.b = cc.b; pend1.h = cc.h;
                        pend1.c_first = c_first; pend1.armed = true;
                    }
                } else {
                    __threadfence();
                    __syncwarp();
                    const int k = (int)((uint32_t)w - c_first);          // this contributor's index in the pair
                    const int ck = (k / kMmaChunk) * kMmaChunk;          // its chunk's first index
                    const uint32_t cw = c_first + (uint32_t)ck;          // chunk's first worker
                    const int first_rec = (ck == 0) ? first_odd : 0;
                    const int n_chunks = (n_parts + kMmaChunk - 1) / kMmaChunk;
                    // first round: chunk level; second round: pair level
                    int32_t* tk = p.counters2 + 2 * cw + first_rec;
                    int n = min(kMmaChunk, n_parts - ck);
                    uint32_t fw = cw;
                    int step = 1, fslot = first_rec;
                    for (int round = 0; round < 2; ++round) {
                        int ticket = 0;
                        if (lane == 0) ticket = atomicAdd(tk, 1);
                        ticket = __shfl_sync(FULL, ticket, 0);
                        if (ticket != n - 1) break;          // someone else arrives later and merges
                        __threadfence();
                        merge_records(n, fw, step, fslot);
                        if (lane == 0) *tk = 0;              // ready for the next launch
                        if (round == 1) { write_rows(cc.b, cc.h); break; }
                        // the chunk's result becomes the record of the chunk's first worker
                        store_record(p.partials + (size_t)(2 * cw + first_rec) * REC);
                        __threadfence();
                        __syncwarp();
                        tk = p.counters + c_first; n = n_chunks; fw = c_first; step = kMmaChunk; fslot = first_odd;
                    }
                }
            }
            m_run[0] = m_run[1] = -INFINITY;
            l_run[0] = l_run[1] = 0.f;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) o[mt][i] = 0.f;
        }
        if (!last) {
            if (pair_end) {
                cc = cn;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) { qb[ks][0] = qn[ks][0]; qb[ks][1] = qn[ks][1]; }
                seg_t0 = 0; cur = nxt; first_seg = false;
            } else {
                rcursor_next(cc, p, H, mp.groups_per_kv, R);
            }
        }
    }

    // The tickets posted above: whoever finds itself the last contributor of a pair merges it.
    if (ok) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const Pending& pd = i == 0 ? pend0 : pend1;
            if (!pd.armed) continue;
            const int ticket = __shfl_sync(FULL, pd.ticket, 0);
            if (ticket != pd.n - 1) continue;            // someone else arrives later and merges
            merge_records(pd.n, pd.c_first, 1, pd.first_odd);
            if (lane == 0) p.counters[pd.c_first] = 0;   // ready for the next launch
            write_rows(pd.b, pd.h);
        }
    }

    if (!ok) {
        if (lane == 0) atomicExch(p.status, kStatusTimeout);
        for (int s = 0; s < NS; ++s) {
            mbar_wait_bounded(bars + 8 * s, 0, 1u << 10);
            mbar_wait_bounded(bars + 8 * s, 1, 1u << 10);
        }
    }
}

}  // namespace lckv
