// Decode attention, FP32-ALU kernel: one query head per (sequence, head) pair.
//
// This is the kernel for multi-head attention (group size 1, 1 flop per KV byte): the work is
// streaming K and V rows from HBM, so it is organised around keeping many bulk copies in flight.
//
//  * A launch is one long sequence of tiles (R cache rows of one (b, head) pair; see plan_kernel),
//    cut into equal contiguous ranges, one per WORKER.  A worker is one warp: it owns a private
//    ring of shared-memory slots, issues its own 1-D bulk (TMA) copies K-tile, V-tile, K-tile, ...
//    into the ring (lane 0), waits on the slot's mbarrier, and consumes the rows with plain FP32
//    FMAs.  No block-level synchronisation exists after start-up.
//  * Softmax is the running-max form (fp32, base-2 exponentials); the state (m, l, o[D]) lives in
//    registers across the tiles of a pair.
//  * A pair that falls entirely inside one worker's range is normalised and written directly.
//    A pair cut by a range boundary leaves an fp32 partial (m, l, o) per contributing worker; the
//    contributor that arrives last (atomic ticket, no waiting) merges them with the log-sum-exp
//    rule in a fixed order and writes the row.  A worker posts its ticket when its part is done
//    but looks at the answer only after its last tile, so the round trip of the atomic and the merge
//    itself never sit between two tiles of its range.
#pragma once
#include "lckv_small_kernels.cuh"

namespace lckv {

// Tuning knobs (compile-time): workers per CTA, ring slots per worker, packed fp32x2 FMAs.
#ifndef LCKV_ALU_WARPS
#define LCKV_ALU_WARPS 8
#endif
#ifndef LCKV_ALU_SLOT_BYTES
#define LCKV_ALU_SLOT_BYTES 8192
#endif
#ifndef LCKV_ALU_SLOTS
#define LCKV_ALU_SLOTS 2
#endif
#ifndef LCKV_ALU_FFMA2
#define LCKV_ALU_FFMA2 1
#endif
#ifndef LCKV_ALU_CTAS
#define LCKV_ALU_CTAS 1
#endif
constexpr int kAluWarps = LCKV_ALU_WARPS;  // workers per CTA
constexpr int kAluCtas = LCKV_ALU_CTAS;    // CTAs per SM (workers never synchronise: any split of an SM's workers into CTAs works)
constexpr int kAluSlots = LCKV_ALU_SLOTS;  // ring slots per worker
constexpr int kAluSlotBytes = LCKV_ALU_SLOT_BYTES;  // one tile of K or of V (a multiple of 4 KB)
constexpr int kAluSmemBytes = kAluWarps * kAluSlots * (kAluSlotBytes + 8);
constexpr int kAluTreeMin = 24;   // pairs split over more workers than this are merged in two levels
constexpr int kAluChunk = 16;     // contributors per first-level chunk

struct AttnParams {
    const uint16_t* K;        // [B_max, H_kv, T_cap, D] bf16
    const uint16_t* V;
    const uint16_t* q;        // [B, H_q, D] bf16
    void* out;                // [B, H_q, D] bf16 or fp32
    float* lse;               // [B, H_q] or null
    const int32_t* lens;      // [B]
    const uint32_t* pre;      // [B + 1] tile prefix for this mode
    const WorkerStart* start; // [n_workers] for this mode: where each worker's range begins
    float* partials;          // [2 * n_workers][D + 4]
    int32_t* counters;        // [n_workers], zero between launches
    int32_t* counters2;      // [2 * n_workers] tickets of first-level merge chunks (tensor-core kernel; may be null)
    int32_t* status;          // device status word
    int64_t T_cap;
    int32_t B, H_q, H_kv, mode, n_workers, out_f32;
    float scale_log2;         // softmax scale * log2(e)
    const int32_t* page_table; // paged caches: [B_max][pt_stride] page ids (shared by all slots), else null
    int32_t pt_stride;        // page-table entries per sequence
    int32_t page_shift;       // log2(rows per page)
    float l2_keep;            // fraction of the cache lines to keep in L2 for the next layer's
                              // pass over the same cache (0: stream everything)
    uint32_t wait_limit;      // polls a wait on a copy may take before the kernel gives up
                              // (status word = timeout, bounded drain, return)
    int32_t early_kv;         // 1: the launcher guarantees that the plan tables and the visible K/V
                              // rows were final before the PREVIOUS kernel in the stream started,
                              // so the first copies may be issued before the dependency wait
};

struct TileCursor {
    int32_t b, h;
    uint32_t t, nt;   // tile within the pair; tiles per pair of sequence b
    int32_t nv;       // visible rows of sequence b
    uint32_t pre0;    // tiles (per pair index) of the sequences before b
};

__device__ __forceinline__ void cursor_load(TileCursor& c, const AttnParams& p)
{
    c.pre0 = __ldg(p.pre + c.b);
    c.nt = __ldg(p.pre + c.b + 1) - c.pre0;
    c.nv = visible_rows(__ldg(p.lens + c.b), p.mode, p.T_cap);
}

// Next tile in (b, pair, tile) order, skipping sequences without tiles.  Safe past the end.
__device__ __forceinline__ void cursor_next(TileCursor& c, const AttnParams& p, int H)
{
    if (++c.t < c.nt) return;
    c.t = 0;
    if (++c.h < H) return;
    c.h = 0;
    do {
        if (++c.b >= p.B) { c.b = p.B; c.nt = 0; c.nv = 0; return; }
        cursor_load(c, p);
    } while (c.nt == 0);
}

// Paged caches: a slot is [n_pages, H_kv, page_rows, D]; logical row r of sequence b lives in page
// page_table[b][r / page_rows].  A tile never straddles pages (page_rows is a multiple of the tile).
// The walker keeps the current page id and prefetches the next one, so the table look-up is off
// the copy-issue path except at the first tile of a sequence.
struct PageWalker {
    int32_t b = -1, pg = -1, id = 0, next = 0;
    __device__ __forceinline__ int64_t row(const AttnParams& p, int bb, int kvh, int r0)
    {
        const int q = r0 >> p.page_shift;
        if (bb != b || q != pg) {
            const int32_t* t = p.page_table + (size_t)bb * p.pt_stride;
            id = (bb == b && q == pg + 1) ? next : __ldg(t + q);
            next = (q + 1 < p.pt_stride) ? __ldg(t + q + 1) : 0;
            b = bb;
            pg = q;
        }
        return (((int64_t)id * p.H_kv + kvh) << p.page_shift) + (r0 & ((1 << p.page_shift) - 1));
    }
};

template <int D, bool PAGED = false>
__global__ void __launch_bounds__(kAluWarps * 32, kAluCtas) attn_alu_kernel(const AttnParams p)
{
    constexpr int SUB = kAluSlotBytes / 4096;   // 4 KB sub-tiles per tile
    constexpr int R1 = 4096 / (D * 2);          // rows per sub-tile: 16 (D=128), 32 (D=64)
    constexpr int R = SUB * R1;                 // rows per tile
    constexpr int LPR = D / 8;                  // lanes per row (16 bytes each)
    constexpr int RPI = 32 / LPR;               // rows covered by one warp-wide 16-byte load
    constexpr int NP = R1 / RPI;                // such loads per sub-tile = partial sums per lane
    constexpr int DUP = LPR / NP;               // lanes that end up holding the same score
    constexpr int NS = kAluSlots;
    constexpr int REC = D + 4;                  // floats per partial record
    static_assert(NP == 8 && (DUP == 1 || DUP == 2), "layout assumes 8 partial sums per lane");

    extern __shared__ __align__(128) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int w = blockIdx.x * kAluWarps + warp;
    const int H = p.H_q;
    const int g = p.H_q / p.H_kv;
    const uint32_t FULL = 0xffffffffu;

    const uint32_t ring = smem_u32(smem) + warp * (NS * kAluSlotBytes);
    const uint32_t bars = smem_u32(smem) + kAluWarps * NS * kAluSlotBytes + warp * (NS * 8);
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
    TileCursor cc;
    cc.b = ws.b; cc.h = ws.h; cc.t = ws.t; cc.nt = ws.nt; cc.nv = ws.nv; cc.pre0 = ws.pre0;
    const uint32_t n_items = 2 * n_tiles;
    TileCursor ci = cc;

    const uint64_t l2pol = make_l2_policy(p.l2_keep);
    PageWalker walker;
    uint32_t issued = 0, islot = 0;
    auto issue = [&]() {
        const int rows = min(R, ci.nv - (int)ci.t * R);
        const uint32_t bytes = (uint32_t)rows * (D * 2);
        const uint16_t* base = (issued & 1) ? p.V : p.K;
        int64_t first_row;
        if constexpr (PAGED)
            first_row = walker.row(p, ci.b, ci.h / g, (int)ci.t * R);
        else
            first_row = ((int64_t)ci.b * p.H_kv + ci.h / g) * p.T_cap + (int64_t)ci.t * R;
        const uint16_t* src = base + first_row * D;
        if (lane == 0) {
            mbar_expect_tx(bars + 8 * islot, bytes);
            bulk_g2s_hint(ring + islot * kAluSlotBytes, src, bytes, bars + 8 * islot, l2pol);
        }
        if (issued & 1) cursor_next(ci, p, H);
        ++issued;
        islot = (islot + 1 == NS) ? 0 : islot + 1;
    };
    {
        const uint32_t pro = n_items < (uint32_t)NS ? n_items : (uint32_t)NS;
        while (issued < pro) issue();
    }
    if (p.early_kv) pdl_wait_then_release();

    // Rows that see nothing (diagonal-masked first token): the zero dummy KV gives o = 0, lse = 0.
    for (int b = in_range ? w : p.B; b < p.B; b += p.n_workers) {
        if (visible_rows(__ldg(p.lens + b), p.mode, p.T_cap) == 0) {
            const int esz = p.out_f32 ? 4 : 2;
            const int n16 = H * D * esz / 16;
            uint4* o16 = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.out) +
                                                  (size_t)b * H * D * esz);
            for (int i = lane; i < n16; i += 32) o16[i] = make_uint4(0, 0, 0, 0);
            if (p.lse)
                for (int i = lane; i < H; i += 32) p.lse[(size_t)b * H + i] = 0.f;
        }
    }

    if (!has_work) return;

    const int grp = lane / LPR;  // which of the RPI rows of a load this lane reads
    const int a = lane % LPR;    // which 16 bytes of the row
    uint32_t cslot = 0, cphase = 0;
    bool ok = true;

    float qf[8];
#if LCKV_ALU_FFMA2
    uint64_t q2[4];   // the same eight values as fp32 pairs
    uint64_t o2[4];   // output accumulators as fp32 pairs (o[] is filled from them at the end)
#pragma unroll
    for (int j = 0; j < 4; ++j) o2[j] = 0ull;
#endif
    auto set_q = [&](const uint4 raw) {
        qf[0] = bf16lo(raw.x) * p.scale_log2; qf[1] = bf16hi(raw.x) * p.scale_log2;
        qf[2] = bf16lo(raw.y) * p.scale_log2; qf[3] = bf16hi(raw.y) * p.scale_log2;
        qf[4] = bf16lo(raw.z) * p.scale_log2; qf[5] = bf16hi(raw.z) * p.scale_log2;
        qf[6] = bf16lo(raw.w) * p.scale_log2; qf[7] = bf16hi(raw.w) * p.scale_log2;
#if LCKV_ALU_FFMA2
#pragma unroll
        for (int j = 0; j < 4; ++j) q2[j] = pack_f32x2(qf[2 * j], qf[2 * j + 1]);
#endif
    };
    set_q(__ldg(reinterpret_cast<const uint4*>(p.q + ((size_t)cc.b * H + cc.h) * D) + a));
    uint32_t seg_t0 = cc.t;
    float m_run = -INFINITY, l_run = 0.f;
    float o[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) o[k] = 0.f;

    // Tickets posted for the (at most two) pairs this worker shares with others: the pair its range
    // starts in the middle of (record 0) and the pair it ends in the middle of (record 1).
    struct Pending { int32_t ticket, n, first_odd, b, h; uint32_t c_first; bool armed; };
    Pending pend0 = {0, 0, 0, 0, 0, 0u, false}, pend1 = pend0;
    // Which workers share a pair: worked out when the worker enters a pair that its range cuts (at
    // most its first and its last), so that the divisions are off the path that ends the kernel.
    struct Split { uint32_t c_first; int32_t n_parts, first_odd; };
    auto split_of = [&](const TileCursor& c) {
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
    float l_tot = 0.f, m_fin = 0.f;   // with o[]: the (unnormalised) result being stored or merged

    // o / l_tot, lse from (m_fin, l_tot) -> output row of pair (b, h)
    auto write_row = [&](int b, int h) {
        const float inv = 1.0f / l_tot;
        const size_t row = (size_t)b * H + h;
        if (lane < LPR) {
            if (p.out_f32) {
                float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.out) + row * D);
                dst[2 * lane] = make_float4(o[0] * inv, o[1] * inv, o[2] * inv, o[3] * inv);
                dst[2 * lane + 1] = make_float4(o[4] * inv, o[5] * inv, o[6] * inv, o[7] * inv);
            } else {
                uint4 pk;
                pk.x = pack_bf16x2(o[0] * inv, o[1] * inv);
                pk.y = pack_bf16x2(o[2] * inv, o[3] * inv);
                pk.z = pack_bf16x2(o[4] * inv, o[5] * inv);
                pk.w = pack_bf16x2(o[6] * inv, o[7] * inv);
                reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + row * D)[lane] = pk;
            }
        }
        if (p.lse && lane == 0) p.lse[row] = (m_fin + lg2(l_tot)) * 0.6931471805599453f;
    };
    // (o, m_fin, l_tot) -> a partial record
    auto store_record = [&](float* rec) {
        if (lane < LPR) {
            reinterpret_cast<float4*>(rec)[2 * lane] = make_float4(o[0], o[1], o[2], o[3]);
            reinterpret_cast<float4*>(rec)[2 * lane + 1] = make_float4(o[4], o[5], o[6], o[7]);
        }
        if (lane == 0) { rec[D] = m_fin; rec[D + 1] = l_tot; }
    };
    // Merge of n records in a fixed order, in one pass with a running maximum: record i is the one of
    // worker first_w + i * step (its second record if i == 0 and first_slot is set).  Record
    // addresses do not depend on loaded data, so the unrolled loop keeps several L2 round trips in
    // flight.  Leaves the merged (unnormalised) values in o, l_tot, m_fin.
    auto merge_records = [&](int n, uint32_t first_w, int step, int first_slot) {
        const float* rec0 = p.partials + (size_t)(2 * first_w) * REC;
        const size_t rstride = (size_t)(2 * step) * REC;
        float M = -INFINITY, Lsum = 0.f, acc[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = 0.f;
#pragma unroll 4
        for (int i = 0; i < n; ++i) {
            const float* r = rec0 + (size_t)i * rstride + (i == 0 ? (size_t)first_slot * REC : 0);
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(r + D));
            float4 x0 = make_float4(0.f, 0.f, 0.f, 0.f), x1 = x0;
            if (lane < LPR) {
                x0 = __ldcg(reinterpret_cast<const float4*>(r) + 2 * lane);
                x1 = __ldcg(reinterpret_cast<const float4*>(r) + 2 * lane + 1);
            }
            const float Mn = fmaxf(M, ml.x);
            const float ca = ex2(M - Mn), cb = ex2(ml.x - Mn);   // ex2(-inf) = 0 for the first record
            M = Mn;
            Lsum = fmaf(Lsum, ca, ml.y * cb);
            acc[0] = fmaf(acc[0], ca, x0.x * cb); acc[1] = fmaf(acc[1], ca, x0.y * cb);
            acc[2] = fmaf(acc[2], ca, x0.z * cb); acc[3] = fmaf(acc[3], ca, x0.w * cb);
            acc[4] = fmaf(acc[4], ca, x1.x * cb); acc[5] = fmaf(acc[5], ca, x1.y * cb);
            acc[6] = fmaf(acc[6], ca, x1.z * cb); acc[7] = fmaf(acc[7], ca, x1.w * cb);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) o[k] = acc[k];
        l_tot = Lsum;
        m_fin = M;
    };

    for (uint32_t tile = 0; tile < n_tiles; ++tile) {
        const int rows = min(R, cc.nv - (int)cc.t * R);
        const bool pair_end = (cc.t + 1 == cc.nt);
        const bool last = (tile + 1 == n_tiles);
        // the next pair's query is fetched while this pair's last tile is worked on
        TileCursor cn = cc;
        uint4 q_next = make_uint4(0, 0, 0, 0);
        if (pair_end && !last) {
            cursor_next(cn, p, H);
            if (n_tiles - (tile + 1) < cn.nt) nxt = split_of(cn);   // the range ends inside the next pair
            q_next = __ldg(reinterpret_cast<const uint4*>(p.q + ((size_t)cn.b * H + cn.h) * D) + a);
        }

        // ---- K tile: scores -----------------------------------------------------------------
        if (!mbar_wait_bounded(bars + 8 * cslot, cphase, p.wait_limit)) { ok = false; break; }
        float part[SUB][NP];
#pragma unroll
        for (int u = 0; u < SUB; ++u) {
            const uint32_t base = ring + cslot * kAluSlotBytes + u * 4096 + grp * (D * 2) + a * 16;
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const uint4 kv = lds128(base + i * (RPI * D * 2));
#if LCKV_ALU_FFMA2
                uint64_t acc = fmul2(pack_f32x2(bf16lo(kv.x), bf16hi(kv.x)), q2[0]);
                acc = ffma2(pack_f32x2(bf16lo(kv.y), bf16hi(kv.y)), q2[1], acc);
                acc = ffma2(pack_f32x2(bf16lo(kv.z), bf16hi(kv.z)), q2[2], acc);
                acc = ffma2(pack_f32x2(bf16lo(kv.w), bf16hi(kv.w)), q2[3], acc);
                float ax, ay;
                unpack_f32x2(acc, ax, ay);
                part[u][i] = ax + ay;
#else
                float s = bf16lo(kv.x) * qf[0];
                s = fmaf(bf16hi(kv.x), qf[1], s);
                s = fmaf(bf16lo(kv.y), qf[2], s);
                s = fmaf(bf16hi(kv.y), qf[3], s);
                s = fmaf(bf16lo(kv.z), qf[4], s);
                s = fmaf(bf16hi(kv.z), qf[5], s);
                s = fmaf(bf16lo(kv.w), qf[6], s);
                s = fmaf(bf16hi(kv.w), qf[7], s);
                part[u][i] = s;
#endif
            }
        }
        __syncwarp();
        if (issued < n_items) issue();  // refill the slot just read
        cslot = (cslot + 1 == NS) ? 0 : cslot + 1;
        if (cslot == 0) cphase ^= 1;

        // Sum each row's LPR partial dot products.  Exchange steps halve the number of values a
        // lane carries (8 -> 4 -> 2 -> 1); with 16 lanes per row one plain butterfly step remains.
        // Afterwards this lane holds, per sub-tile, the score of load index a / DUP, i.e. of row:
        const int my_row = (a / DUP) * RPI + grp;
        float sc[SUB];
#pragma unroll
        for (int u = 0; u < SUB; ++u) {
            float* pt = part[u];
            bool up = (a & (LPR / 2)) != 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float send = up ? pt[k] : pt[k + 4];
                const float keep = up ? pt[k + 4] : pt[k];
                pt[k] = keep + __shfl_xor_sync(FULL, send, LPR / 2);
            }
            up = (a & (LPR / 4)) != 0;
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const float send = up ? pt[k] : pt[k + 2];
                const float keep = up ? pt[k + 2] : pt[k];
                pt[k] = keep + __shfl_xor_sync(FULL, send, LPR / 4);
            }
            up = (a & (LPR / 8)) != 0;
            {
                const float send = up ? pt[0] : pt[1];
                const float keep = up ? pt[1] : pt[0];
                pt[0] = keep + __shfl_xor_sync(FULL, send, LPR / 8);
            }
            if (DUP == 2) pt[0] += __shfl_xor_sync(FULL, pt[0], 1);
            sc[u] = (u * R1 + my_row < rows) ? pt[0] : -INFINITY;
        }

        float m_tile = sc[0];
#pragma unroll
        for (int u = 1; u < SUB; ++u) m_tile = fmaxf(m_tile, sc[u]);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1)
            m_tile = fmaxf(m_tile, __shfl_xor_sync(FULL, m_tile, off));
        const float m_new = fmaxf(m_run, m_tile);
        const float alpha = ex2(m_run - m_new);
        float pr[SUB];
        float p_sum = 0.f;
#pragma unroll
        for (int u = 0; u < SUB; ++u) {
            pr[u] = ex2(sc[u] - m_new);
            p_sum += pr[u];
        }
        l_run = fmaf(l_run, alpha, p_sum);
        m_run = m_new;
#if LCKV_ALU_FFMA2
        {
            const uint64_t a2 = pack_f32x2(alpha, alpha);
#pragma unroll
            for (int j = 0; j < 4; ++j) o2[j] = fmul2(o2[j], a2);
        }
#else
#pragma unroll
        for (int k = 0; k < 8; ++k) o[k] *= alpha;
#endif

        // ---- V tile: weighted sum -----------------------------------------------------------
        if (!mbar_wait_bounded(bars + 8 * cslot, cphase, p.wait_limit)) { ok = false; break; }
        if (rows < R) {
            // Rows past the copy hold leftovers of an earlier tile; their weight is 0 but 0 * NaN
            // is NaN, so clear them.  Generic-proxy writes, fenced before the slot's next copy.
            const uint32_t vb = ring + cslot * kAluSlotBytes;
            for (int i = rows * (D * 2) + lane * 16; i < R * D * 2; i += 32 * 16)
                sts128(vb + i, make_uint4(0, 0, 0, 0));
            fence_proxy_async_smem();
            __syncwarp();
        }
#pragma unroll
        for (int u = 0; u < SUB; ++u) {
            const uint32_t base = ring + cslot * kAluSlotBytes + u * 4096 + grp * (D * 2) + a * 16;
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const float pi = __shfl_sync(FULL, pr[u], grp * LPR + i * DUP);
                const uint4 vv = lds128(base + i * (RPI * D * 2));
#if LCKV_ALU_FFMA2
                const uint64_t p2 = pack_f32x2(pi, pi);
                o2[0] = ffma2(p2, pack_f32x2(bf16lo(vv.x), bf16hi(vv.x)), o2[0]);
                o2[1] = ffma2(p2, pack_f32x2(bf16lo(vv.y), bf16hi(vv.y)), o2[1]);
                o2[2] = ffma2(p2, pack_f32x2(bf16lo(vv.z), bf16hi(vv.z)), o2[2]);
                o2[3] = ffma2(p2, pack_f32x2(bf16lo(vv.w), bf16hi(vv.w)), o2[3]);
#else
                o[0] = fmaf(pi, bf16lo(vv.x), o[0]);
                o[1] = fmaf(pi, bf16hi(vv.x), o[1]);
                o[2] = fmaf(pi, bf16lo(vv.y), o[2]);
                o[3] = fmaf(pi, bf16hi(vv.y), o[3]);
                o[4] = fmaf(pi, bf16lo(vv.z), o[4]);
                o[5] = fmaf(pi, bf16hi(vv.z), o[5]);
                o[6] = fmaf(pi, bf16lo(vv.w), o[6]);
                o[7] = fmaf(pi, bf16hi(vv.w), o[7]);
#endif
            }
        }
        __syncwarp();
        if (issued < n_items) issue();
        cslot = (cslot + 1 == NS) ? 0 : cslot + 1;
        if (cslot == 0) cphase ^= 1;

        // ---- end of this worker's part of the pair? -----------------------------------------
        if (pair_end || last) {
            // everything this worker saw of the pair: reduce over row groups and lanes
#if LCKV_ALU_FFMA2
#pragma unroll
            for (int j = 0; j < 4; ++j) unpack_f32x2(o2[j], o[2 * j], o[2 * j + 1]);
#endif
#pragma unroll
            for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
                for (int k = 0; k < 8; ++k) o[k] += __shfl_xor_sync(FULL, o[k], off);
            l_tot = l_run;
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) l_tot += __shfl_xor_sync(FULL, l_tot, off);
            l_tot *= (1.0f / DUP);
            m_fin = m_run;

            const bool complete = pair_end && seg_t0 == 0;
            if (complete) {
                write_row(cc.b, cc.h);
            } else {
                const uint32_t c_first = cur.c_first;
                const int first_odd = cur.first_odd, n_parts = cur.n_parts;
                const bool at_lo = first_seg;
                store_record(p.partials + (size_t)(2 * w + (at_lo ? 0 : 1)) * REC);
                // Few parts: the contributor that arrives last merges them all.  Many parts (few
                // pairs, long sequences): two levels - the contributors of a pair form chunks of
                // kAluChunk consecutive workers; the last arriver of a chunk merges the chunk's records
                // into the record of the chunk's first worker, and the last chunk to finish merges
                // the chunk records.  Same fixed order either way.
                const bool two_level = n_parts > kAluTreeMin && p.counters2 != nullptr;
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
                    const int kk = (int)((uint32_t)w - c_first);         // this contributor's index in the pair
                    const int ck = (kk / kAluChunk) * kAluChunk;         // its chunk's first index
                    const uint32_t cw = c_first + (uint32_t)ck;          // chunk's first worker
                    const int first_rec = (ck == 0) ? first_odd : 0;
                    int32_t* tk = p.counters2 + 2 * cw + first_rec;
                    int n = min(kAluChunk, n_parts - ck);
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
                        if (round == 1) { write_row(cc.b, cc.h); break; }
                        // the chunk's result becomes the record of the chunk's first worker
                        store_record(p.partials + (size_t)(2 * cw + first_rec) * REC);
                        __threadfence();
                        __syncwarp();
                        tk = p.counters + c_first; n = (n_parts + kAluChunk - 1) / kAluChunk; fw = c_first;
                        step = kAluChunk; fslot = first_odd;
                    }
                }
            }
            m_run = -INFINITY;
            l_run = 0.f;
#pragma unroll
            for (int k = 0; k < 8; ++k) o[k] = 0.f;
#if LCKV_ALU_FFMA2
#pragma unroll
            for (int j = 0; j < 4; ++j) o2[j] = 0ull;
#endif
        }
        if (!last) {
            cc = pair_end ? cn : cc;
            if (pair_end) { set_q(q_next); seg_t0 = 0; cur = nxt; first_seg = false; }
            else cursor_next(cc, p, H);
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
            write_row(pd.b, pd.h);
        }
    }

    if (!ok) {
        // A copy never landed.  Report it, give the copies still in flight a bounded chance to
        // finish (they target this CTA's shared memory), and leave.
        if (lane == 0) atomicExch(p.status, kStatusTimeout);
        for (int s = 0; s < NS; ++s) {
            mbar_wait_bounded(bars + 8 * s, 0, 1u << 10);
            mbar_wait_bounded(bars + 8 * s, 1, 1u << 10);
        }
    }
}

}  // namespace lckv
