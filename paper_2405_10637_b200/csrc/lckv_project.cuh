// Fused K/V producer: k = x W_K^T, v = x W_V^T for the new token of every sequence, written
// straight into row len[b] of a cache slot (paper Section 2.1: only the layers that own a cache
// still compute K and V; W_K, W_V are the maps from hidden states to keys and values).
//
// The contraction runs on the 5th-generation tensor cores with the operands swapped, so that the
// 128 rows of the MMA tile are output features (one head at d_h = 128, two at d_h = 64) and the
// batch is the N side (16 ... 256): small decode batches do not pad a 128-row tile.
//
//   D^T [128 features x NB sequences] = W [128 x d_model] . x^T [d_model x NB]
//
//   warp 0     producer: 2-D TMA loads of the W tile [128 x 64 k_boxes] and the x tile [NB x 64 k_boxes]
//              per k-step (boxes of 64 columns = one 128-byte swizzled row each)
//   warp 1     one thread issues tcgen05.mma (both operands K-major in shared memory, fp32
//              accumulator in tensor memory); tcgen05.commit frees the stage / signals the end
//   warps 2-5  epilogue: tensor memory -> fp32 staging in shared memory (the pipeline's stages,
//              idle by then), optional rotation of the key by its position (half-split pairs
//              d, d + d_h/2 with caller-provided cos / sin tables), one rounding to bf16,
//              16-byte stores into the cache row (ring position and page look-up as in
//              append_kernel).
//
// Small batches are bound by streaming the weights, and a layer has only (2 H_kv d_h / 128) feature
// tiles - 64 at the 7B width, fewer than the SMs.  The launch may therefore split d_model over a
// thread-block cluster of k_split CTAs (cluster dimension z): each CTA accumulates its share of the
// k-steps, all write their fp32 tile to their own shared memory, and each CTA finishes a share of
// the tile's columns, adding the other CTAs' partial values through distributed shared memory
// (two cluster barriers: tiles written / tiles read).  The rotation tables must be 16-byte aligned.
//
// The launch carries the programmatic-serialization attribute.  The weights never depend on the
// kernel before this one in the stream, so a CTA fills its pipeline with W tiles first and only
// then executes griddepcontrol.wait; x, the lengths, the page table, the rotation tables, the cache
// rows and the status word are touched after that wait.  A CTA lets its own dependents be scheduled
// once it has requested its last bytes, so that a dependent with the same habit streams its first
// weights while this kernel runs its epilogue.
//
// Every wait is bounded; a wait that runs out sets the status word and the kernel returns.
#pragma once
#include "lckv_prefill_tc5.cuh"

namespace lckv {

constexpr int kProjThreads = 192;
constexpr int kProjBM = 128;            // output features per CTA
constexpr int kProjBoxCols = 64;        // d_model columns per TMA box (one 128-byte swizzled row); a k-step is
                                        // k_boxes such boxes requested together, so that a weight row is
                                        // fetched in runs of k_boxes * 128 contiguous bytes
constexpr int kProjPad = 4;             // fp32 padding of a staged column (keeps 16-byte alignment)
constexpr uint32_t kProjWaitLimit = 1u << 16;
constexpr int kProjColGroup = 4;        // columns whose lengths / pages / rotation factors are fetched together

struct ProjParams {
    uint16_t* K;              // slot's K and V tensors (contiguous or paged pool)
    uint16_t* V;
    const int32_t* lens;      // [B] tokens cached so far = position of the new token
    const float* rope_cos;    // [rope_positions, D/2] or null
    const float* rope_sin;
    int32_t* status;
    const int32_t* page_table;
    int64_t T_cap;
    int32_t pt_stride, page_shift;
    int32_t B, H_kv, D, d_model;
    int32_t NB;               // batch tile = N of the MMA (a multiple of 16, at most 256)
    int32_t n_stages;
    int32_t n_sink;
    int32_t k_tiles;          // feature tiles of K; tiles k_tiles .. 2*k_tiles-1 belong to V
    int32_t rope_positions;
    int32_t k_split;          // CTAs of a cluster that share one tile's k-steps (1, 2, 4, 8)
    int32_t k_boxes;          // 64-column boxes per k-step (1, 2, 4)
};

__host__ __device__ inline int proj_stage_bytes(int NB, int k_boxes) { return (kProjBM + NB) * 128 * k_boxes; }
__host__ __device__ inline int proj_smem_bytes(int NB, int n_stages, int k_boxes)
{
    const int pipe = n_stages * proj_stage_bytes(NB, k_boxes);
    const int stage_out = NB * (kProjBM + kProjPad) * 4;
    return (pipe > stage_out ? pipe : stage_out) + 256 + 1024;
}

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Hardware barrier over all threads of the cluster (every thread of every CTA executes it).
__device__ __forceinline__ void cluster_sync_all()
{
    __syncwarp();
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
// 16 bytes of another CTA's shared memory: `addr` is the address in this CTA's own window.
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr, uint32_t rank)
{
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(addr), "r"(rank));
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(ra)
                 : "memory");
    return v;
}

__global__ void __launch_bounds__(kProjThreads)
project_kv_kernel(const ProjParams p, const __grid_constant__ CUtensorMap tmX,
                  const __grid_constant__ CUtensorMap tmWk, const __grid_constant__ CUtensorMap tmWv)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int NB = p.NB, NS = p.n_stages;
    const int KB = p.k_boxes, BK = kProjBoxCols * KB;
    const int w_bytes = kProjBM * 128 * KB;
    const int stage_bytes = proj_stage_bytes(NB, KB);
    const int pipe = NS * stage_bytes;
    const int stage_out = NB * (kProjBM + kProjPad) * 4;
    const uint32_t bars = smem0 + (uint32_t)(pipe > stage_out ? pipe : stage_out);
    // barriers: full[s] at bars + 8 s, empty[s] at bars + 96 + 8 s (s < 12), accumulator at +192
    const uint32_t bFull = bars, bEmpty = bars + 96, bAcc = bars + 192, sTaddr = bars + 200;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mt = blockIdx.x;                 // feature tile
    const int b0 = blockIdx.y * NB;            // first sequence of the batch tile
    const bool is_v = mt >= p.k_tiles;
    const int f0 = (is_v ? mt - p.k_tiles : mt) * kProjBM;   // first feature within K or V
    const int KS = p.k_split;
    const uint32_t rank = KS > 1 ? cluster_ctarank() : 0u;
    const int n_k = (p.d_model + BK - 1) / BK / KS;   // this CTA's k-steps (columns past d_model read as zero)
    const int k_first = (int)rank * n_k;
    uint32_t tm_cols = 32;                      // allocation: a power of two >= NB
    while ((int)tm_cols < NB) tm_cols *= 2;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(bFull + 8 * s, 1); mbar_init(bEmpty + 8 * s, 1); }
        mbar_init(bAcc, 1);
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(sTaddr, tm_cols);
    tc5_fence_before();
    __syncthreads();
    tc5_fence_after();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(sTaddr));

    bool ok = true;
    // Epilogue threads: what a column needs from global memory (the sequence's length, its page, the
    // rotation factors at its position), fetched for kProjColGroup columns at a time so that the
    // round trips overlap; the first group is fetched while the weights still stream.
    struct ColPre { int32_t t; int64_t dst_row; float4 c0, c1, s0, s1; };
    ColPre cp[kProjColGroup];
    const int e_t = tid - 64;                               // 0..127 in the epilogue warps
    const int e_per = NB / KS;                              // columns this CTA finishes
    const int e_lo = (int)rank * e_per, e_hi = e_lo + e_per;
    const int e_fl = (e_t & 15) * 8;                        // first of this thread's 8 features in the tile
    const int e_kvh = (f0 + e_fl) / p.D, e_d = (f0 + e_fl) - e_kvh * p.D;
    const bool e_rot = (!is_v) && p.rope_cos != nullptr;
    auto fetch_cols = [&](int col0) {
        const int half = p.D >> 1, i0 = e_d < half ? e_d : e_d - half;
#pragma unroll
        for (int u = 0; u < kProjColGroup; ++u) {
            const int col = col0 + 8 * u, b = b0 + col;
            cp[u].t = (col < e_hi && b < p.B) ? __ldg(p.lens + b) : -1;
        }
#pragma unroll
        for (int u = 0; u < kProjColGroup; ++u) {
            const int col = col0 + 8 * u, b = b0 + col;
            const int32_t t = cp[u].t;
            int64_t row = t;
            if (p.n_sink > 0 && row >= p.T_cap) row = p.n_sink + (row - p.n_sink) % (p.T_cap - p.n_sink);
            cp[u].dst_row = -1;                                  // (the host refuses calls with rows out of range)
            if (row < 0 || row >= p.T_cap) continue;
            cp[u].dst_row = ((int64_t)b * p.H_kv + e_kvh) * p.T_cap + row;
            if (p.page_table) {
                const int64_t id = __ldg(p.page_table + (int64_t)b * p.pt_stride + (row >> p.page_shift));
                cp[u].dst_row = ((id * p.H_kv + e_kvh) << p.page_shift) + (row & ((1 << p.page_shift) - 1));
            }
            if (e_rot) {
                const int pos = t < p.rope_positions ? t : p.rope_positions - 1;  // host checks the range
                const float4* cs4 = reinterpret_cast<const float4*>(p.rope_cos + (size_t)pos * half + i0);
                const float4* sn4 = reinterpret_cast<const float4*>(p.rope_sin + (size_t)pos * half + i0);
                cp[u].c0 = __ldg(cs4); cp[u].c1 = __ldg(cs4 + 1);
                cp[u].s0 = __ldg(sn4); cp[u].s1 = __ldg(sn4 + 1);
            }
        }
    };
    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const void* tmW = is_v ? (const void*)&tmWv : (const void*)&tmWk;
            // The pipeline's first fill: weights before the dependency wait, x after it.
            const int pro = n_k < NS ? n_k : NS;
            for (int k = 0; k < pro; ++k) {
                mbar_expect_tx(bFull + 8 * k, (uint32_t)stage_bytes);
                for (int j = 0; j < KB; ++j)
                    tma_load_2d(smem0 + k * stage_bytes + j * (kProjBM * 128), tmW, (k_first + k) * BK + j * 64,
                                f0, bFull + 8 * k);
            }
            pdl_wait();
            for (int k = 0; k < pro; ++k)
                for (int j = 0; j < KB; ++j)
                    tma_load_2d(smem0 + k * stage_bytes + w_bytes + j * (NB * 128), &tmX,
                                (k_first + k) * BK + j * 64, b0, bFull + 8 * k);
            for (int k = pro; k < n_k && ok; ++k) {
                const int s = k % NS;
                ok = mbar_wait_bounded(bEmpty + 8 * s, ((k / NS) - 1) & 1, kProjWaitLimit);
                if (!ok) break;
                const uint32_t dst = smem0 + s * stage_bytes;
                mbar_expect_tx(bFull + 8 * s, (uint32_t)stage_bytes);
                for (int j = 0; j < KB; ++j)
                    tma_load_2d(dst + j * (kProjBM * 128), tmW, (k_first + k) * BK + j * 64, f0, bFull + 8 * s);
                for (int j = 0; j < KB; ++j)
                    tma_load_2d(dst + w_bytes + j * (NB * 128), &tmX, (k_first + k) * BK + j * 64, b0,
                                bFull + 8 * s);
            }
            // This CTA has asked for its last bytes: from here on a dependent kernel may be scheduled
            // beside it, so that the dependent's own first weights stream while this kernel finishes.
            pdl_release();
            if (!ok) atomicExch(p.status, kStatusTimeout);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = tc5_idesc(kProjBM, NB, 0);
            pdl_wait();   // (a timeout below writes the status word)
            for (int k = 0; k < n_k && ok; ++k) {
                const int s = k % NS;
                ok = mbar_wait_bounded(bFull + 8 * s, (k / NS) & 1, kProjWaitLimit);
                if (!ok) break;
                tc5_fence_after();
                const uint32_t a0 = smem0 + s * stage_bytes, x0 = a0 + w_bytes;
                for (int j = 0; j < KB; ++j)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        tc5_mma(tmem_base, tc5_desc(a0 + j * (kProjBM * 128) + ks * 32, 16, 1024),
                                tc5_desc(x0 + j * (NB * 128) + ks * 32, 16, 1024), idesc, (k > 0 || j > 0 || ks > 0));
                tc5_commit(bEmpty + 8 * s);
            }
            if (ok) tc5_commit(bAcc);
            else atomicExch(p.status, kStatusTimeout);
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int q4 = warp & 3;
        const int r = q4 * 32 + lane;                       // feature row of the tile = TMEM lane
        const uint32_t lane_sel = (uint32_t)(q4 * 32) << 16;
        const int ld = kProjBM + kProjPad;
        pdl_wait();   // before the lengths, the page table and the cache rows are touched
        fetch_cols(e_lo + (e_t >> 4));
        ok = mbar_wait_bounded(bAcc, 0, kProjWaitLimit);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc5_fence_after();
            // accumulator -> staging [col][feature] fp32 (all MMAs are done: the stages are free)
            for (int c0 = 0; c0 < NB; c0 += 32) {
                uint32_t v[32];
                // NB = 16: the allocation still has 32 columns; the upper 16 are read and dropped
                tmem_ld32(tmem_base + lane_sel + c0, v);
                const int nc = NB - c0 < 32 ? NB - c0 : 32;
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    if (c < nc)
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(smem0 + (uint32_t)(((c0 + c) * ld + r) * 4)),
                                     "r"(v[c]) : "memory");
            }
        } else if (lane == 0) {
            atomicExch(p.status, kStatusTimeout);
        }
    }

    // All tiles of the cluster are in their CTAs' staging areas (or a wait ran out and the status
    // word says so); every thread of every CTA reaches the barriers below.
    tc5_fence_before();
    __syncthreads();
    if (KS > 1) cluster_sync_all();

    if (warp >= 2) {
        const int et = tid - 64;                            // 0..127
        const int ld = kProjBM + kProjPad;
        float* stg = reinterpret_cast<float*>(smem_raw + (smem0 - smem_u32(smem_raw)));
        // The CTAs of a cluster share the columns: rank r finishes columns [c_lo, c_hi).
        const int per = NB / KS;
        const int c_lo = (int)rank * per, c_hi = c_lo + per;
        if (ok && KS > 1) {
            // Pass 1: add the other CTAs' partial values of these columns into this CTA's staging
            // (independent 16-byte loads through distributed shared memory, several in flight).
            const int n4 = per * ld / 4;
            float4* mine = reinterpret_cast<float4*>(stg + c_lo * ld);
            const uint32_t a0 = smem0 + (uint32_t)(c_lo * ld * 4);
            for (int i0 = et; i0 < n4; i0 += 128 * 4) {
                float4 acc[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + 128 * u;
                    acc[u] = i < n4 ? mine[i] : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                for (int rk = 0; rk < KS; ++rk) {
                    if (rk == (int)rank) continue;
                    float4 rv[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int i = i0 + 128 * u;
                        rv[u] = i < n4 ? ld_cluster_f4(a0 + (uint32_t)i * 16, (uint32_t)rk)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        acc[u].x += rv[u].x; acc[u].y += rv[u].y; acc[u].z += rv[u].z; acc[u].w += rv[u].w;
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + 128 * u;
                    if (i < n4) mine[i] = acc[u];
                }
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");   // all four epilogue warps, whatever ok says
        if (ok) {
            // Pass 2: rotation, rounding, stores - from this CTA's shared memory only.
            const int half = p.D >> 1;
            const int fl = e_fl, d = e_d;
            const int fl_partner = d < half ? fl + half : fl - half;
            const float sgn = d < half ? -1.f : 1.f;
            uint16_t* base = is_v ? p.V : p.K;
            for (int col0 = c_lo + (et >> 4); col0 < c_hi; col0 += 8 * kProjColGroup) {
                if (col0 != c_lo + (et >> 4)) fetch_cols(col0);   // the first group is in registers already
#pragma unroll
                for (int u = 0; u < kProjColGroup; ++u) {
                    const int col = col0 + 8 * u;
                    if (col >= c_hi || cp[u].dst_row < 0) continue;
                    float x[8];
                    {
                        const float4 lo = *reinterpret_cast<const float4*>(stg + col * ld + fl);
                        const float4 hi = *reinterpret_cast<const float4*>(stg + col * ld + fl + 4);
                        x[0] = lo.x; x[1] = lo.y; x[2] = lo.z; x[3] = lo.w;
                        x[4] = hi.x; x[5] = hi.y; x[6] = hi.z; x[7] = hi.w;
                    }
                    if (e_rot) {
                        const float4 pl = *reinterpret_cast<const float4*>(stg + col * ld + fl_partner);
                        const float4 ph = *reinterpret_cast<const float4*>(stg + col * ld + fl_partner + 4);
                        const float xp[8] = {pl.x, pl.y, pl.z, pl.w, ph.x, ph.y, ph.z, ph.w};
                        const float4 c0 = cp[u].c0, c1 = cp[u].c1, s0 = cp[u].s0, s1 = cp[u].s1;
                        const float cs[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
                        const float sn[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
                        for (int i = 0; i < 8; ++i) x[i] = fmaf(sgn * xp[i], sn[i], x[i] * cs[i]);
                    }
                    const uint4 packed = make_uint4(cvt_bf16x2(x[0], x[1]), cvt_bf16x2(x[2], x[3]),
                                                    cvt_bf16x2(x[4], x[5]), cvt_bf16x2(x[6], x[7]));
                    *reinterpret_cast<uint4*>(base + cp[u].dst_row * p.D + d) = packed;
                }
            }
        }
    }

    // a CTA's shared memory must outlive the other CTAs' reads
    if (KS > 1) cluster_sync_all();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, tm_cols);
}

}  // namespace lckv
