// Host runtime and C ABI of the LCKV decode-attention library (see include/lckv.h).
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/lckv.h"
#include "lckv_attn_alu.cuh"
#include "lckv_attn_mma.cuh"
#include "lckv_project.cuh"
#include "lckv_prefill.cuh"
#include "lckv_prefill_tc5.cuh"
#include "lckv_probe.cuh"
#include "lckv_small_kernels.cuh"

namespace {

thread_local int g_last_cuda_error = 0;

inline bool cuda_ok(cudaError_t e)
{
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return false;
    }
    return true;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Host-side layer plan; the rule is stated in the header (Section 2.1 of the paper).
struct Plan {
    std::vector<int32_t> is_warmup, read_slot, mode, write_slot, write_before;
    int32_t n_slots = 0;
};

int make_plan(int L, int w, int variant, Plan& pl)
{
    if (L < 1 || w < 0 || w > L) return LCKV_EINVAL;
    if (w != L && (w & 1)) return LCKV_EINVAL;
    if (variant != 0 && variant != 1) return LCKV_EINVAL;
    pl.is_warmup.assign(L, 0);
    pl.read_slot.assign(L, 0);
    pl.mode.assign(L, LCKV_MODE_CONDENSED);
    pl.write_slot.assign(L, -1);
    pl.write_before.assign(L, 0);
    const int half = w / 2;
    for (int l = 0; l < L; ++l) pl.is_warmup[l] = (w == L) || l < half || l >= L - half;
    // The layer whose k,v fill slot 0.
    const int feeder = (variant == 1 && w > 0 && w < L) ? L - 1 - half : L - 1;
    int next_slot = 1;
    for (int l = 0; l < L; ++l) {
        if (pl.is_warmup[l]) {
            const int s = (l == feeder) ? 0 : next_slot++;
            pl.read_slot[l] = pl.write_slot[l] = s;
            pl.mode[l] = LCKV_MODE_STANDARD;
            pl.write_before[l] = 1;
        } else if (l == feeder) {
            pl.write_slot[l] = 0;
        }
    }
    pl.n_slots = next_slot;
    return LCKV_OK;
}

struct Layout {
    size_t off_pt;
    size_t off_lens, off_pre, off_start, off_counters, off_status, off_partials, off_slots;
    size_t off_stage_q, off_stage_out, off_stage_kv;
    size_t slot_bytes, workspace_bytes, total_bytes;
    size_t stage_q_bytes, stage_out_bytes, stage_kv_bytes;  // per layer
    int pre_stride;
};

}  // namespace

struct lckv_cache {
    lckv_config_t cfg;
    Plan plan;
    Layout lay;
    float scale_log2;
    int sm_count, n_workers, grid, rows_per_tile, h_pairs, kernel_kind;
    int active_workers;                   // workers a launch uses (<= n_workers; lckv_cache_set_worker_limit)
    uint8_t* base;
    int32_t* d_lens;
    uint32_t* d_pre;
    lckv::WorkerStart* d_start;
    int32_t* d_counters;
    int32_t* d_status;
    float* d_partials;
    std::vector<int32_t> h_lens;  // host mirror of the device lengths
    int n_kv_layers;
    std::vector<CUtensorMap> tm_k, tm_v;  // per slot, tensor-core kernel only
    std::vector<CUtensorMap> tm_pf_k, tm_pf_v;  // per slot, 64-row boxes for prompt encoding
    // paged caches (cfg.page_rows > 0): page table mirror and the pool's free list
    int pt_stride, page_shift;
    int32_t* d_pt;
    std::vector<int32_t> h_pt;            // [max_batch][pt_stride], -1 = none
    std::vector<int32_t> n_pages_of;      // pages held per sequence
    std::vector<int32_t> free_pages;      // stack of free page ids
    bool pt_dirty;
    int prefill_tc5;                      // 1: prompt encoding on tcgen05, 0: mma.sync kernel
    double l2_keep_bytes;                 // how much of a re-read slot to hold in L2 (0 = off)
    uint32_t wait_limit;                  // polls a device-side wait on a copy may take
    int ws_parity;                        // which half of the split-K workspace the next launch uses
    size_t partials_half_floats;          // floats in one half of the partial records
    // CUDA graph of one step, valid for the argument pointers it was captured with
    // Captured steps, most recently used first: a caller that alternates between a few sets of
    // buffers (double-buffered activations) replays instead of re-capturing.
    struct CapturedStep { std::vector<const void*> key; cudaGraphExec_t exec; };
    std::vector<CapturedStep> graphs;
    // host-buffer step: copy streams and events (created on first use when cfg.host_staging)
    cudaStream_t s_in = nullptr, s_out = nullptr;
    std::vector<cudaEvent_t> ev;          // [0] step start, [1] k/v in, [2] all out, then per chunk in / done
    // descriptors of the producer's operands (x, W_K, W_V), keyed by address and shape
    struct OperandMap { const void* ptr; uint64_t rows, cols; int box_rows; CUtensorMap tm; };
    std::vector<OperandMap> operand_maps;
};

namespace {

int validate_config(const lckv_config_t* c)
{
    if (!c || c->struct_size != sizeof(lckv_config_t)) return LCKV_EINVAL;
    if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1) return LCKV_EINVAL;
    if (c->n_q_heads % c->n_kv_heads) return LCKV_EINVAL;
    if (c->head_dim != 64 && c->head_dim != 128) return LCKV_EINVAL;
    if (c->max_batch < 1 || c->max_seq < 1) return LCKV_EINVAL;
    if (!(c->softmax_scale >= 0.f) || !std::isfinite(c->softmax_scale)) return LCKV_EINVAL;
    if (c->out_dtype != 0 && c->out_dtype != 1) return LCKV_EINVAL;
    if (c->kernel_kind != 0 && c->kernel_kind != 1) return LCKV_EINVAL;
    if (c->stream_sink < 0 || (c->stream_sink > 0 && c->stream_sink >= c->max_seq)) return LCKV_EINVAL;
    if (c->page_rows != 0) {
        const int P = c->page_rows;
        if (P < 64 || P > 65536 || (P & (P - 1)) || c->n_pages < 1 || c->stream_sink > 0) return LCKV_EINVAL;
    }
    Plan pl;
    if (int rc = make_plan(c->n_layers, c->n_warmup, c->top_variant, pl)) return rc;
    // tile counts are kept in 32 bits
    const uint64_t tiles = (uint64_t)c->max_batch * (((uint64_t)c->max_seq + 15) / 16);
    if (tiles >= (1ull << 31)) return LCKV_EINVAL;
    return LCKV_OK;
}

// 1 = FP32-ALU kernel, 2 = tensor-core kernel (query groups of 2 ... 7 and multiples of 8).
int resolve_kernel_kind(const lckv_config_t& c)
{
    const int g = c.n_q_heads / c.n_kv_heads;
    // the tensor-core kernel addresses cache rows through 32-bit TMA coordinates
    const uint64_t rows = c.page_rows ? (uint64_t)c.n_pages * c.n_kv_heads * (uint64_t)c.page_rows
                                      : (uint64_t)c.max_batch * c.n_kv_heads * (uint64_t)c.max_seq;
    // groups of 8 fill the N = 8 side of the MMA tile; smaller groups (2 ... 7) use it with the
    // remaining columns zero, which still reads K and V once per group instead of once per head
    const bool fits = g % 8 == 0 || (g >= 2 && g < 8);
    return (c.kernel_kind == 0 && fits && rows < (1ull << 31)) ? 2 : 1;
}

// Query heads per pair of the tensor-core kernel: 8, or the whole group when it is smaller.
int mma_heads_per_pair(const lckv_config_t& c)
{
    const int g = c.n_q_heads / c.n_kv_heads;
    return g < 8 ? g : 8;
}

int workers_per_sm(const lckv_config_t& c)
{
    return resolve_kernel_kind(c) == 2 ? lckv::kMmaWarps * lckv::kMmaCtas : lckv::kAluWarps * lckv::kAluCtas;
}

int partial_record_floats(const lckv_config_t& c)
{
    return resolve_kernel_kind(c) == 2 ? c.head_dim * 8 + 16 : c.head_dim + 4;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of one K or V tensor seen as [rows = B_max*H_kv*T_cap, d_h] bf16, box = 64 columns x
// `box_rows` rows, 128-byte swizzle, out-of-range rows read as zero.
int make_tensor_map_pitch(CUtensorMap* tm, void* base, uint64_t rows, uint64_t cols,
                          uint64_t pitch_bytes, int box_rows);

int make_tensor_map(CUtensorMap* tm, void* base, uint64_t rows, int d, int box_rows)
{
    return make_tensor_map_pitch(tm, base, rows, (uint64_t)d, (uint64_t)d * 2, box_rows);
}

// General form: a bf16 matrix of `rows` x `cols` with a row pitch in bytes (multiple of 16).
int make_tensor_map_pitch(CUtensorMap* tm, void* base, uint64_t rows, uint64_t cols,
                          uint64_t pitch_bytes, int box_rows)
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (!cuda_ok(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q)))
            return LCKV_ECUDA;
        if (q != cudaDriverEntryPointSuccess || !f) return LCKV_ECUDA;
        fn = reinterpret_cast<EncodeTiledFn>(f);
    }
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)pitch_bytes};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = (int)r;
        return LCKV_ECUDA;
    }
    return LCKV_OK;
}

void make_layout(const lckv_config_t& c, int n_slots, int n_workers, int n_kv_layers, Layout& y)
{
    const size_t A = 256;
    size_t off = 0;
    y.off_lens = off;      off = align_up(off + (size_t)c.max_batch * 4, A);
    y.pre_stride = (int)align_up((size_t)c.max_batch + 1, 64);
    y.off_pre = off;       off = align_up(off + 2 * (size_t)y.pre_stride * 4, A);
    y.off_start = off;     off = align_up(off + 2 * (size_t)n_workers * sizeof(lckv::WorkerStart), A);
    y.off_counters = off;  off = align_up(off + 2 * 3 * (size_t)n_workers * 4, A);  // two halves of [pair tickets | chunk tickets]
    y.off_status = off;    off = align_up(off + 4, A);
    y.off_partials = off;
    off = align_up(off + 2 * 2 * (size_t)n_workers * partial_record_floats(c) * 4, A);  // two halves
    y.slot_bytes =
        c.page_rows ? align_up((size_t)c.n_pages * c.n_kv_heads * (size_t)c.page_rows * c.head_dim * 2, A)
                    : align_up((size_t)c.max_batch * c.n_kv_heads * (size_t)c.max_seq * c.head_dim * 2, A);
    y.off_pt = off;
    if (c.page_rows)
        off = align_up(off + (size_t)c.max_batch * ((c.max_seq + c.page_rows - 1) / c.page_rows) * 4, A);
    y.workspace_bytes = off;
    y.off_slots = off;     off += 2 * (size_t)n_slots * y.slot_bytes;
    y.stage_q_bytes = align_up((size_t)c.max_batch * c.n_q_heads * c.head_dim * 2, A);
    y.stage_out_bytes =
        align_up((size_t)c.max_batch * c.n_q_heads * c.head_dim * (c.out_dtype ? 4 : 2), A);
    y.stage_kv_bytes = align_up((size_t)c.max_batch * c.n_kv_heads * c.head_dim * 2, A);
    y.off_stage_q = y.off_stage_out = y.off_stage_kv = 0;
    if (c.host_staging) {
        y.off_stage_q = off;    off += (size_t)c.n_layers * y.stage_q_bytes;
        y.off_stage_out = off;  off += (size_t)c.n_layers * y.stage_out_bytes;
        y.off_stage_kv = off;   off += 2 * (size_t)n_kv_layers * y.stage_kv_bytes;
    }
    y.total_bytes = off;
}

int device_sm_count(int* sm)
{
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return LCKV_ECUDA;
    if (!cuda_ok(cudaDeviceGetAttribute(sm, cudaDevAttrMultiProcessorCount, dev))) return LCKV_ECUDA;
    return LCKV_OK;
}

uint16_t* slot_k(const lckv_cache* c, int s)
{
    return reinterpret_cast<uint16_t*>(c->base + c->lay.off_slots + (size_t)(2 * s) * c->lay.slot_bytes);
}
uint16_t* slot_v(const lckv_cache* c, int s)
{
    return reinterpret_cast<uint16_t*>(c->base + c->lay.off_slots +
                                       (size_t)(2 * s + 1) * c->lay.slot_bytes);
}

// Longest sequence, for capacity checks; 0 in streaming mode (a ring never overflows).
int max_len(const lckv_cache* c, int batch)
{
    if (c->cfg.stream_sink > 0) return 0;
    int m = 0;
    for (int b = 0; b < batch; ++b) m = c->h_lens[b] > m ? c->h_lens[b] : m;
    return m;
}

// Paged caches: make sure every sequence b < batch owns pages for h_lens[b] + extra rows, taking
// pages from the pool.  On exhaustion nothing is changed and LCKV_ECAPACITY is returned.
int ensure_pages(lckv_cache* c, int batch, int extra)
{
    if (!c->cfg.page_rows) return LCKV_OK;
    std::vector<std::pair<int, int>> taken;  // (sequence, page) for roll-back
    for (int b = 0; b < batch; ++b) {
        const int rows = c->h_lens[b] + extra;
        if (rows > c->cfg.max_seq) break;  // reported by the caller's own capacity check
        const int need = (rows + c->cfg.page_rows - 1) >> c->page_shift;
        while (c->n_pages_of[b] < need) {
            if (c->free_pages.empty()) {
                for (auto it = taken.rbegin(); it != taken.rend(); ++it) {
                    c->free_pages.push_back(it->second);
                    c->h_pt[(size_t)it->first * c->pt_stride + --c->n_pages_of[it->first]] = -1;
                }
                return LCKV_ECAPACITY;
            }
            const int pg = c->free_pages.back();
            c->free_pages.pop_back();
            c->h_pt[(size_t)b * c->pt_stride + c->n_pages_of[b]++] = pg;
            taken.emplace_back(b, pg);
        }
    }
    if (!taken.empty()) c->pt_dirty = true;
    return LCKV_OK;
}

// Paged caches, on reset: sequences b < batch give their pages back and get ceil(len / P) new ones.
// Checked first, so that a pool too small for the request changes nothing.
int repage(lckv_cache* c, const int32_t* lens, int batch)
{
    if (!c->cfg.page_rows) return LCKV_OK;
    size_t need = 0, held = 0;
    for (int b = 0; b < batch; ++b) {
        const int rows = lens ? lens[b] : 0;
        if (rows > c->cfg.max_seq) return LCKV_ECAPACITY;
        need += (size_t)((rows + c->cfg.page_rows - 1) >> c->page_shift);
        held += (size_t)c->n_pages_of[b];
    }
    if (need > c->free_pages.size() + held) return LCKV_ECAPACITY;
    for (int b = 0; b < batch; ++b) {
        while (c->n_pages_of[b] > 0) {
            int32_t& e = c->h_pt[(size_t)b * c->pt_stride + --c->n_pages_of[b]];
            c->free_pages.push_back(e);
            e = -1;
        }
    }
    for (int b = 0; b < batch; ++b) {
        const int rows = lens ? lens[b] : 0;
        const int n = (rows + c->cfg.page_rows - 1) >> c->page_shift;
        for (int i = 0; i < n; ++i) {
            c->h_pt[(size_t)b * c->pt_stride + i] = c->free_pages.back();
            c->free_pages.pop_back();
        }
        c->n_pages_of[b] = n;
    }
    c->pt_dirty = true;
    return LCKV_OK;
}

// Upload the page table if it changed since the last upload (pageable source: staged before return).
int sync_page_table(lckv_cache* c, cudaStream_t st)
{
    if (!c->cfg.page_rows || !c->pt_dirty) return LCKV_OK;
    if (!cuda_ok(cudaMemcpyAsync(c->d_pt, c->h_pt.data(), c->h_pt.size() * 4, cudaMemcpyHostToDevice, st)))
        return LCKV_ECUDA;
    c->pt_dirty = false;
    return LCKV_OK;
}

int launch_plan(lckv_cache* c, int batch, cudaStream_t st)
{
    lckv::plan_kernel<<<1, 1024, 0, st>>>(c->d_lens, batch, c->rows_per_tile, c->h_pairs,
                                          c->active_workers, c->d_pre, c->lay.pre_stride, c->d_start,
                                          c->cfg.max_seq);
    return cuda_ok(cudaGetLastError()) ? LCKV_OK : LCKV_ECUDA;
}

// Launch with the programmatic-serialization attribute: the kernel may be scheduled while its
// predecessor in the stream drains; it orders itself with griddepcontrol.wait.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st,
                       Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// early: the previous kernel in the stream is an attention launch of the same step and this one
// reads only rows that were final before it (condensed mode), so its first copies need not wait.
int launch_attention(lckv_cache* c, int slot, int mode, const void* q, void* out, float* lse,
                     int batch, cudaStream_t st, bool early = false, float l2_keep = 0.f)
{
    lckv::AttnParams p;
    p.K = slot_k(c, slot);
    p.V = slot_v(c, slot);
    p.q = static_cast<const uint16_t*>(q);
    p.out = out;
    p.lse = lse;
    p.lens = c->d_lens;
    p.pre = c->d_pre + (size_t)mode * c->lay.pre_stride;
    p.start = c->d_start + (size_t)mode * c->active_workers;   // (the plan kernel's stride)
    // consecutive launches may overlap at their edges: alternate the split-K workspace halves
    p.partials = c->d_partials + (size_t)c->ws_parity * c->partials_half_floats;
    p.counters = c->d_counters + (size_t)c->ws_parity * 3 * c->n_workers;
    p.counters2 = p.counters + c->n_workers;
    c->ws_parity ^= 1;
    p.status = c->d_status;
    p.T_cap = c->cfg.max_seq;
    p.B = batch;
    p.H_q = c->cfg.n_q_heads;
    p.H_kv = c->cfg.n_kv_heads;
    p.mode = mode;
    p.n_workers = c->active_workers;
    p.out_f32 = c->cfg.out_dtype;
    p.scale_log2 = c->scale_log2;
    p.early_kv = early ? 1 : 0;
    p.wait_limit = c->wait_limit;
    p.l2_keep = l2_keep;
    p.page_table = c->d_pt;
    p.pt_stride = c->pt_stride;
    p.page_shift = c->page_shift;
    const bool paged = c->cfg.page_rows != 0;
    cudaError_t e;
    if (c->kernel_kind == 2) {
        lckv::MmaParams mp;
        mp.a = p;
        mp.a.H_q = c->h_pairs;  // pairs per sequence = groups of up to 8 query heads
        mp.n_q_heads = c->cfg.n_q_heads;
        mp.heads_per_pair = mma_heads_per_pair(c->cfg);
        mp.groups_per_kv = c->cfg.n_q_heads / c->cfg.n_kv_heads / mp.heads_per_pair;
        const int blk = lckv::kMmaWarps * 32;
        const size_t sm = lckv::kMmaSmemBytes;
        if (c->cfg.head_dim == 128)
            e = paged ? launch_pdl(lckv::attn_mma_kernel<128, true>, c->grid, blk, sm, st, mp, c->tm_k[slot], c->tm_v[slot])
                      : launch_pdl(lckv::attn_mma_kernel<128, false>, c->grid, blk, sm, st, mp, c->tm_k[slot], c->tm_v[slot]);
        else
            e = paged ? launch_pdl(lckv::attn_mma_kernel<64, true>, c->grid, blk, sm, st, mp, c->tm_k[slot], c->tm_v[slot])
                      : launch_pdl(lckv::attn_mma_kernel<64, false>, c->grid, blk, sm, st, mp, c->tm_k[slot], c->tm_v[slot]);
    } else {
        const int blk = lckv::kAluWarps * 32;
        const size_t sm = lckv::kAluSmemBytes;
        if (c->cfg.head_dim == 128)
            e = paged ? launch_pdl(lckv::attn_alu_kernel<128, true>, c->grid, blk, sm, st, p)
                      : launch_pdl(lckv::attn_alu_kernel<128, false>, c->grid, blk, sm, st, p);
        else
            e = paged ? launch_pdl(lckv::attn_alu_kernel<64, true>, c->grid, blk, sm, st, p)
                      : launch_pdl(lckv::attn_alu_kernel<64, false>, c->grid, blk, sm, st, p);
    }
    return cuda_ok(e) ? LCKV_OK : LCKV_ECUDA;
}

int launch_append(lckv_cache* c, int slot, const void* k_new, const void* v_new, int batch,
                  cudaStream_t st)
{
    const int64_t n = (int64_t)batch * c->cfg.n_kv_heads * (c->cfg.head_dim / 8);
    const int threads = 256;
    const int blocks = (int)((n + threads - 1) / threads);
    lckv::append_kernel<<<blocks, threads, 0, st>>>(
        slot_k(c, slot), slot_v(c, slot), static_cast<const uint16_t*>(k_new),
        static_cast<const uint16_t*>(v_new), c->d_lens, batch, c->cfg.n_kv_heads, c->cfg.max_seq,
        c->cfg.head_dim, c->cfg.stream_sink, c->d_pt, c->pt_stride, c->page_shift);
    return cuda_ok(cudaGetLastError()) ? LCKV_OK : LCKV_ECUDA;
}

int launch_advance(lckv_cache* c, int batch, cudaStream_t st)
{
    lckv::advance_kernel<<<(batch + 255) / 256, 256, 0, st>>>(c->d_lens, batch);
    return cuda_ok(cudaGetLastError()) ? LCKV_OK : LCKV_ECUDA;
}

void mirror_advance(lckv_cache* c, int batch)
{
    for (int b = 0; b < batch; ++b) c->h_lens[b] += 1;
}

// Fraction of a re-read slot's lines to mark evict-last, judged from the host mirror of the
// lengths, in sixteenths (so that a captured step stays valid while the caches grow a little).
float step_keep_frac(const lckv_cache* c, int batch)
{
    int64_t rows = 0;
    for (int b = 0; b < batch; ++b)
        rows += c->h_lens[b] < c->cfg.max_seq ? c->h_lens[b] : c->cfg.max_seq;
    const double bytes = (double)rows * 4.0 * c->cfg.n_kv_heads * c->cfg.head_dim;
    if (bytes <= 0 || c->l2_keep_bytes <= 0) return 0.f;
    const double f = std::fmin(1.0, c->l2_keep_bytes / bytes);
    return (float)(std::floor(f * 16.0) / 16.0);
}

// The launches of one step, in the order the header states.
// Events around layers of a step (host-buffer step: inputs arrive and outputs leave on other streams).
struct StepHooks {
    std::vector<cudaEvent_t> wait_before;   // per layer: wait for this event before the layer (or null)
    std::vector<cudaEvent_t> record_after;  // per layer: record this event after the layer (or null)
};

int enqueue_step(lckv_cache* c, const void* const* q, void* const* out, const void* const* kn,
                 const void* const* vn, int batch, cudaStream_t st, const StepHooks* hooks = nullptr)
{
    const Plan& pl = c->plan;
    const int L = c->cfg.n_layers;
    // A step starts after fully serialised launches (advance, plan), so it may always begin with
    // workspace half 0; this also makes a captured step replayable.
    c->ws_parity = 0;
    if (int rc = launch_plan(c, batch, st)) return rc;
    // A slot that several layers read in this step is worth keeping in L2 between their passes, as
    // far as it fits: mark that fraction of its lines evict-last.  A slot read once is streamed.
    const float keep_frac = step_keep_frac(c, batch);
    std::vector<int> readers(pl.n_slots, 0);
    for (int l = 0; l < L; ++l) readers[pl.read_slot[l]] += 1;
    bool prev_attn = false;
    for (int l = 0; l < L; ++l) {
        if (hooks && hooks->wait_before[l]) {
            if (!cuda_ok(cudaStreamWaitEvent(st, hooks->wait_before[l], 0))) return LCKV_ECUDA;
            prev_attn = false;   // the launch that follows an event wait waits in full
        }
        if (pl.write_slot[l] >= 0 && pl.write_before[l]) {
            if (int rc = launch_append(c, pl.write_slot[l], kn[l], vn[l], batch, st)) return rc;
            prev_attn = false;
        }
        const bool early = prev_attn && pl.mode[l] == LCKV_MODE_CONDENSED;
        const float keep = readers[pl.read_slot[l]] > 1 ? keep_frac : 0.f;
        if (int rc = launch_attention(c, pl.read_slot[l], pl.mode[l], q[l], out[l], nullptr, batch,
                                      st, early, keep))
            return rc;
        prev_attn = true;
        if (hooks && hooks->record_after[l]) {
            if (!cuda_ok(cudaEventRecord(hooks->record_after[l], st))) return LCKV_ECUDA;
            prev_attn = false;
        }
    }
    for (int l = 0; l < L; ++l)
        if (pl.write_slot[l] >= 0 && !pl.write_before[l])
            if (int rc = launch_append(c, pl.write_slot[l], kn[l], vn[l], batch, st)) return rc;
    return launch_advance(c, batch, st);
}

constexpr size_t kMaxCapturedSteps = 4;

void drop_graph(lckv_cache* c)
{
    for (auto& g : c->graphs)
        if (g.exec) cudaGraphExecDestroy(g.exec);
    c->graphs.clear();
}

// One step through a CUDA graph, captured the first time a set of argument pointers, batch and kept
// L2 fraction is seen (up to kMaxCapturedSteps sets are remembered).
int step_with_graph(lckv_cache* c, const void* const* q, void* const* out, const void* const* kn,
                    const void* const* vn, int batch, cudaStream_t st)
{
    const int L = c->cfg.n_layers;
    std::vector<const void*> key;
    key.reserve(4 * L + 2);
    key.push_back(reinterpret_cast<const void*>((uintptr_t)batch));
    key.push_back(reinterpret_cast<const void*>((uintptr_t)(step_keep_frac(c, batch) * 16.f)));
    for (int l = 0; l < L; ++l) {
        key.push_back(q[l]);
        key.push_back(out[l]);
        key.push_back(c->plan.write_slot[l] >= 0 ? kn[l] : nullptr);
        key.push_back(c->plan.write_slot[l] >= 0 ? vn[l] : nullptr);
    }
    size_t hit = 0;
    while (hit < c->graphs.size() && c->graphs[hit].key != key) ++hit;
    if (hit == c->graphs.size()) {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (!cuda_ok(cudaStreamIsCapturing(st, &cs))) return LCKV_ECUDA;
        // The caller is capturing already, or the stream is the legacy default stream (which
        // cannot be captured): just issue the launches.
        if (cs != cudaStreamCaptureStatusNone || st == nullptr || st == cudaStreamLegacy)
            return enqueue_step(c, q, out, kn, vn, batch, st);
        if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
            (void)cudaGetLastError();
            return enqueue_step(c, q, out, kn, vn, batch, st);
        }
        const int rc = enqueue_step(c, q, out, kn, vn, batch, st);
        cudaGraph_t g = nullptr;
        const bool ended = cuda_ok(cudaStreamEndCapture(st, &g));
        if (rc || !ended || !g) {
            if (g) cudaGraphDestroy(g);
            return rc ? rc : LCKV_ECUDA;
        }
        cudaGraphExec_t exec = nullptr;
        const bool inst = cuda_ok(cudaGraphInstantiate(&exec, g, 0));
        cudaGraphDestroy(g);
        if (!inst) return LCKV_ECUDA;
        if (c->graphs.size() >= kMaxCapturedSteps) {   // the least recently used one goes
            cudaGraphExecDestroy(c->graphs.back().exec);
            c->graphs.pop_back();
        }
        c->graphs.push_back({key, exec});
        hit = c->graphs.size() - 1;
    }
    if (hit != 0) std::rotate(c->graphs.begin(), c->graphs.begin() + hit, c->graphs.begin() + hit + 1);
    if (!cuda_ok(cudaGraphLaunch(c->graphs.front().exec, st))) return LCKV_ECUDA;
    c->ws_parity = c->cfg.n_layers & 1;  // where the captured step leaves it
    return LCKV_OK;
}

int run_step(lckv_cache* c, const void* const* q, void* const* out, const void* const* kn,
             const void* const* vn, int batch, cudaStream_t st)
{
    if (int rc = ensure_pages(c, batch, 1)) return rc;   // room for this step's token
    if (int rc = sync_page_table(c, st)) return rc;
    const int rc = c->cfg.use_graph ? step_with_graph(c, q, out, kn, vn, batch, st)
                                    : enqueue_step(c, q, out, kn, vn, batch, st);
    if (rc == LCKV_OK) mirror_advance(c, batch);
    return rc;
}

int prefill_check(const lckv_cache* c, int n_max, int batch, bool attention)
{
    if (c->cfg.stream_sink > 0) return LCKV_EINVAL;
    if (attention && c->tm_pf_k.empty()) return LCKV_EINVAL;  // slot too large for 32-bit TMA rows
    if (batch < 1 || batch > c->cfg.max_batch || n_max < 1) return LCKV_EINVAL;
    for (int b = 0; b < batch; ++b)
        if (c->h_lens[b] > n_max) return LCKV_EINVAL;
    return LCKV_OK;
}

int launch_prefill_write(lckv_cache* c, int slot, const void* k, const void* v, int n_max,
                         int batch, cudaStream_t st)
{
    const int64_t n = (int64_t)batch * n_max * c->cfg.n_kv_heads * (c->cfg.head_dim / 8);
    const int threads = 256;
    lckv::prefill_write_kv_kernel<<<(unsigned)((n + threads - 1) / threads), threads, 0, st>>>(
        slot_k(c, slot), slot_v(c, slot), static_cast<const uint16_t*>(k),
        static_cast<const uint16_t*>(v), c->d_lens, batch, n_max, c->cfg.n_kv_heads, c->cfg.max_seq,
        c->cfg.head_dim, c->d_pt, c->pt_stride, c->page_shift);
    return cuda_ok(cudaGetLastError()) ? LCKV_OK : LCKV_ECUDA;
}

int launch_prefill_attention(lckv_cache* c, int slot, int mode, const void* q, void* out,
                             int n_max, int batch, cudaStream_t st)
{
    lckv::PrefillParams p;
    p.q = static_cast<const uint16_t*>(q);
    p.out = out;
    p.lens = c->d_lens;
    p.status = c->d_status;
    p.T_cap = c->cfg.max_seq;
    p.B = batch;
    p.n_max = n_max;
    p.H_q = c->cfg.n_q_heads;
    p.H_kv = c->cfg.n_kv_heads;
    p.mode = mode;
    p.out_f32 = c->cfg.out_dtype;
    p.scale_log2 = c->scale_log2;
    p.page_table = c->d_pt;
    p.pt_stride = c->pt_stride;
    p.page_shift = c->page_shift;
    int longest = 0;
    for (int b = 0; b < batch; ++b) longest = c->h_lens[b] > longest ? c->h_lens[b] : longest;
    if (longest == 0) return LCKV_OK;
    if (c->prefill_tc5) {
        // tcgen05 kernel: 128-row query blocks; the Q tile comes through a tensor map built for this
        // call's q pointer: q seen as [batch * n_max rows, H_q * d_h columns]
        const uint64_t q_rows = (uint64_t)batch * n_max;
        if (q_rows >= (1ull << 31)) return LCKV_EINVAL;
        CUtensorMap tmq;
        if (int rc = make_tensor_map_pitch(&tmq, const_cast<void*>(q), q_rows,
                                           (uint64_t)c->cfg.n_q_heads * c->cfg.head_dim,
                                           (uint64_t)c->cfg.n_q_heads * c->cfg.head_dim * 2, lckv::kT5BM))
            return rc;
        const dim3 grid5((longest + lckv::kT5BM - 1) / lckv::kT5BM, c->cfg.n_q_heads, batch);
        if (c->cfg.head_dim == 128)
            lckv::prefill_tc5_kernel<128><<<grid5, lckv::kT5Threads, lckv::tc5_smem_bytes<128>(), st>>>(
                p, tmq, c->tm_pf_k[slot], c->tm_pf_v[slot]);
        else
            lckv::prefill_tc5_kernel<64><<<grid5, lckv::kT5Threads, lckv::tc5_smem_bytes<64>(), st>>>(
                p, tmq, c->tm_pf_k[slot], c->tm_pf_v[slot]);
        return cuda_ok(cudaGetLastError()) ? LCKV_OK : LCKV_ECUDA;
    }
    const dim3 grid((longest + lckv::kPfBM - 1) / lckv::kPfBM, c->cfg.n_q_heads, batch);
    if (c->cfg.head_dim == 128)
        lckv::prefill_attn_kernel<128><<<grid, lckv::kPfWarps * 32, lckv::prefill_smem_bytes<128>(), st>>>(
            p, c->tm_pf_k[slot], c->tm_pf_v[slot]);
    else
        lckv::prefill_attn_kernel<64><<<grid, lckv::kPfWarps * 32, lckv::prefill_smem_bytes<64>(), st>>>(
            p, c->tm_pf_k[slot], c->tm_pf_v[slot]);
    return cuda_ok(cudaGetLastError()) ? LCKV_OK : LCKV_ECUDA;
}

// Copies `n` equally sized layer buffers between host and the staging area (device pitch
// `dev_pitch`).  When the host buffers are contiguous (one allocation sliced per layer) this is a
// single pitched copy; otherwise, or if that copy is refused, one copy per layer.
int copy_layers(uint8_t* dev, size_t dev_pitch, const void* const* host, int n, size_t bytes,
                bool to_device, cudaStream_t st)
{
    if (n <= 0 || bytes == 0) return LCKV_OK;
    bool contiguous = n >= 2;
    for (int l = 1; l < n && contiguous; ++l)
        contiguous = static_cast<const uint8_t*>(host[l]) ==
                     static_cast<const uint8_t*>(host[l - 1]) + bytes;
    if (contiguous) {
        const cudaError_t e =
            to_device ? cudaMemcpy2DAsync(dev, dev_pitch, host[0], bytes, bytes, n,
                                          cudaMemcpyHostToDevice, st)
                      : cudaMemcpy2DAsync(const_cast<void*>(host[0]), bytes, dev, dev_pitch, bytes, n,
                                          cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) return LCKV_OK;
        (void)cudaGetLastError();  // fall back to per-layer copies
    }
    for (int l = 0; l < n; ++l) {
        const cudaError_t e =
            to_device ? cudaMemcpyAsync(dev + (size_t)l * dev_pitch, host[l], bytes, cudaMemcpyHostToDevice, st)
                      : cudaMemcpyAsync(const_cast<void*>(host[l]), dev + (size_t)l * dev_pitch, bytes,
                                        cudaMemcpyDeviceToHost, st);
        if (!cuda_ok(e)) return LCKV_ECUDA;
    }
    return LCKV_OK;
}

}  // namespace

extern "C" {

int lckv_plan(int32_t n_layers, int32_t n_warmup, int32_t top_variant, int32_t* is_warmup,
              int32_t* read_slot, int32_t* mode, int32_t* write_slot, int32_t* write_before,
              int32_t* n_slots)
{
    if (!is_warmup || !read_slot || !mode || !write_slot || !write_before || !n_slots)
        return LCKV_EINVAL;
    Plan pl;
    if (int rc = make_plan(n_layers, n_warmup, top_variant, pl)) return rc;
    for (int l = 0; l < n_layers; ++l) {
        is_warmup[l] = pl.is_warmup[l];
        read_slot[l] = pl.read_slot[l];
        mode[l] = pl.mode[l];
        write_slot[l] = pl.write_slot[l];
        write_before[l] = pl.write_before[l];
    }
    *n_slots = pl.n_slots;
    return LCKV_OK;
}

size_t lckv_cache_bytes(const lckv_config_t* cfg)
{
    if (validate_config(cfg)) return 0;
    int sm = 0;
    if (device_sm_count(&sm)) return 0;
    Plan pl;
    make_plan(cfg->n_layers, cfg->n_warmup, cfg->top_variant, pl);
    int n_kv = 0;
    for (int l = 0; l < cfg->n_layers; ++l) n_kv += pl.write_slot[l] >= 0;
    Layout y;
    make_layout(*cfg, pl.n_slots, sm * workers_per_sm(*cfg), n_kv, y);
    return y.total_bytes;
}

int lckv_cache_alloc(lckv_cache_t** out, const lckv_config_t* cfg, void* dev_buf, size_t dev_bytes)
{
    if (!out || !dev_buf) return LCKV_EINVAL;
    if (int rc = validate_config(cfg)) return rc;
    if (reinterpret_cast<uintptr_t>(dev_buf) % 256) return LCKV_ENOMEM;
    int sm = 0;
    if (int rc = device_sm_count(&sm)) return rc;
    lckv_cache* c = new (std::nothrow) lckv_cache();
    if (!c) return LCKV_ENOMEM;
    c->cfg = *cfg;
    make_plan(cfg->n_layers, cfg->n_warmup, cfg->top_variant, c->plan);
    c->n_kv_layers = 0;
    for (int l = 0; l < cfg->n_layers; ++l) c->n_kv_layers += c->plan.write_slot[l] >= 0;
    c->sm_count = sm;
    c->grid = sm * (resolve_kernel_kind(*cfg) == 2 ? lckv::kMmaCtas : lckv::kAluCtas);
    c->n_workers = sm * workers_per_sm(*cfg);
    c->active_workers = c->n_workers;
    c->kernel_kind = resolve_kernel_kind(*cfg);
    c->rows_per_tile = (c->kernel_kind == 2 ? lckv::kMmaSlotBytes : lckv::kAluSlotBytes) / (cfg->head_dim * 2);
    c->h_pairs = c->kernel_kind == 2 ? cfg->n_q_heads / mma_heads_per_pair(*cfg) : cfg->n_q_heads;
    make_layout(*cfg, c->plan.n_slots, c->n_workers, c->n_kv_layers, c->lay);
    if (dev_bytes < c->lay.total_bytes) { delete c; return LCKV_ENOMEM; }
    const float scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale
                                                 : 1.0f / std::sqrt((float)cfg->head_dim);
    c->scale_log2 = scale * 1.4426950408889634f;
    c->base = static_cast<uint8_t*>(dev_buf);
    c->d_lens = reinterpret_cast<int32_t*>(c->base + c->lay.off_lens);
    c->d_pre = reinterpret_cast<uint32_t*>(c->base + c->lay.off_pre);
    c->d_start = reinterpret_cast<lckv::WorkerStart*>(c->base + c->lay.off_start);
    c->d_counters = reinterpret_cast<int32_t*>(c->base + c->lay.off_counters);
    c->d_status = reinterpret_cast<int32_t*>(c->base + c->lay.off_status);
    c->d_partials = reinterpret_cast<float*>(c->base + c->lay.off_partials);
    c->h_lens.assign(cfg->max_batch, 0);
    c->pt_stride = c->page_shift = 0;
    c->d_pt = nullptr;
    c->pt_dirty = false;
    if (cfg->page_rows) {
        c->pt_stride = (cfg->max_seq + cfg->page_rows - 1) / cfg->page_rows;
        while ((1 << c->page_shift) < cfg->page_rows) ++c->page_shift;
        c->d_pt = reinterpret_cast<int32_t*>(c->base + c->lay.off_pt);
        c->h_pt.assign((size_t)cfg->max_batch * c->pt_stride, -1);
        c->n_pages_of.assign(cfg->max_batch, 0);
        c->free_pages.resize(cfg->n_pages);
        for (int i = 0; i < cfg->n_pages; ++i) c->free_pages[i] = cfg->n_pages - 1 - i;  // pop gives 0, 1, ...
        c->pt_dirty = true;
    }
    {
        // About half of the L2 (measured optimum on B200, 126 MB L2: 60-70 MB; more than that and
        // the evict-last lines start displacing each other).  LCKV_L2_KEEP_MB overrides (0 = off).
        int dev = 0, l2 = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev);
        const char* env = getenv("LCKV_L2_KEEP_MB");
        c->l2_keep_bytes = env ? atof(env) * 1e6 : 0.52 * (double)l2;
    }
    {
        const char* env = getenv("LCKV_PREFILL_KERNEL");   // "mma" selects the mma.sync kernel
        c->prefill_tc5 = !(env && env[0] == 'm');
    }
    c->ws_parity = 0;
    c->wait_limit = lckv::kDefaultWaitLimit;
    c->partials_half_floats = 2 * (size_t)c->n_workers * partial_record_floats(*cfg);

    if (c->kernel_kind == 2) {
        const uint64_t rows = cfg->page_rows
                                  ? (uint64_t)cfg->n_pages * cfg->n_kv_heads * (uint64_t)cfg->page_rows
                                  : (uint64_t)cfg->max_batch * cfg->n_kv_heads * (uint64_t)cfg->max_seq;
        c->tm_k.resize(c->plan.n_slots);
        c->tm_v.resize(c->plan.n_slots);
        for (int s = 0; s < c->plan.n_slots; ++s) {
            int rc = make_tensor_map(&c->tm_k[s], slot_k(c, s), rows, cfg->head_dim, c->rows_per_tile);
            if (!rc) rc = make_tensor_map(&c->tm_v[s], slot_v(c, s), rows, cfg->head_dim, c->rows_per_tile);
            if (rc) { delete c; return rc; }
        }
    }
    {
        // prompt-encoding kernel: 64-row boxes over every slot (coordinates are 32-bit)
        const uint64_t rows = cfg->page_rows
                                  ? (uint64_t)cfg->n_pages * cfg->n_kv_heads * (uint64_t)cfg->page_rows
                                  : (uint64_t)cfg->max_batch * cfg->n_kv_heads * (uint64_t)cfg->max_seq;
        if (rows < (1ull << 31)) {
            c->tm_pf_k.resize(c->plan.n_slots);
            c->tm_pf_v.resize(c->plan.n_slots);
            for (int s = 0; s < c->plan.n_slots; ++s) {
                int rc = make_tensor_map(&c->tm_pf_k[s], slot_k(c, s), rows, cfg->head_dim, lckv::kPfBN);
                if (!rc) rc = make_tensor_map(&c->tm_pf_v[s], slot_v(c, s), rows, cfg->head_dim, lckv::kPfBN);
                if (rc) { delete c; return rc; }
            }
        }
    }
    bool ok = cuda_ok(cudaFuncSetAttribute(lckv::attn_alu_kernel<128, true>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::kAluSmemBytes)) &&
              cuda_ok(cudaFuncSetAttribute(lckv::attn_alu_kernel<64, true>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::kAluSmemBytes)) &&
              cuda_ok(cudaFuncSetAttribute(lckv::attn_mma_kernel<128, true>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::kMmaSmemBytes)) &&
              cuda_ok(cudaFuncSetAttribute(lckv::attn_mma_kernel<64, true>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::kMmaSmemBytes)) &&
              cuda_ok(cudaFuncSetAttribute(lckv::project_kv_kernel,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           227 * 1024)) &&
              cuda_ok(cudaFuncSetAttribute(lckv::prefill_tc5_kernel<128>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::tc5_smem_bytes<128>())) &&
              cuda_ok(cudaFuncSetAttribute(lckv::prefill_tc5_kernel<64>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::tc5_smem_bytes<64>())) &&
              cuda_ok(cudaFuncSetAttribute(lckv::prefill_attn_kernel<128>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::prefill_smem_bytes<128>())) &&
              cuda_ok(cudaFuncSetAttribute(lckv::prefill_attn_kernel<64>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::prefill_smem_bytes<64>())) &&
              cuda_ok(cudaFuncSetAttribute(lckv::attn_mma_kernel<128>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::kMmaSmemBytes)) &&
              cuda_ok(cudaFuncSetAttribute(lckv::attn_mma_kernel<64>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::kMmaSmemBytes)) &&
              cuda_ok(cudaFuncSetAttribute(lckv::attn_alu_kernel<128>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::kAluSmemBytes)) &&
              cuda_ok(cudaFuncSetAttribute(lckv::attn_alu_kernel<64>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           lckv::kAluSmemBytes)) &&
              cuda_ok(cudaMemset(c->base, 0, c->lay.workspace_bytes)) &&
              cuda_ok(cudaDeviceSynchronize());
    if (!ok) { delete c; return LCKV_ECUDA; }
    *out = c;
    return LCKV_OK;
}

int lckv_cache_free(lckv_cache_t* cache)
{
    if (!cache) return LCKV_EINVAL;
    drop_graph(cache);
    for (cudaEvent_t e : cache->ev) cudaEventDestroy(e);
    if (cache->s_in) cudaStreamDestroy(cache->s_in);
    if (cache->s_out) cudaStreamDestroy(cache->s_out);
    delete cache;
    return LCKV_OK;
}

int lckv_cache_info(const lckv_cache_t* c, lckv_info_t* info)
{
    if (!c || !info) return LCKV_EINVAL;
    info->n_slots = c->plan.n_slots;
    info->n_workers = c->n_workers;
    info->rows_per_tile = c->rows_per_tile;
    info->kernel_kind = c->kernel_kind;
    int launches = 2 + c->cfg.n_layers + c->n_kv_layers;  // plan + advance + attention + appends
    info->launches_per_step = launches;
    info->sm_count = c->sm_count;
    info->slot_bytes = c->lay.slot_bytes;
    info->workspace_bytes = c->lay.workspace_bytes;
    return LCKV_OK;
}

int lckv_cache_reset(lckv_cache_t* c, const int32_t* host_lens, int32_t batch, void* stream)
{
    if (!c || batch < 1 || batch > c->cfg.max_batch) return LCKV_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (host_lens) {
        for (int b = 0; b < batch; ++b) {
            if (host_lens[b] < 0) return LCKV_EINVAL;
            if (host_lens[b] > c->cfg.max_seq && c->cfg.stream_sink == 0) return LCKV_ECAPACITY;
        }
        if (int rc = repage(c, host_lens, batch)) return rc;
        for (int b = 0; b < batch; ++b) c->h_lens[b] = host_lens[b];
        // h_lens is the staging source: it lives as long as the cache and pageable copies are
        // staged before the call returns.
        if (!cuda_ok(cudaMemcpyAsync(c->d_lens, c->h_lens.data(), (size_t)batch * 4,
                                     cudaMemcpyHostToDevice, st)))
            return LCKV_ECUDA;
    } else {
        if (int rc = repage(c, nullptr, batch)) return rc;
        for (int b = 0; b < batch; ++b) c->h_lens[b] = 0;
        if (!cuda_ok(cudaMemsetAsync(c->d_lens, 0, (size_t)batch * 4, st))) return LCKV_ECUDA;
    }
    if (!cuda_ok(cudaMemsetAsync(c->d_counters, 0, 2 * 3 * (size_t)c->n_workers * 4, st))) return LCKV_ECUDA;
    if (!cuda_ok(cudaMemsetAsync(c->d_status, 0, 4, st))) return LCKV_ECUDA;
    return sync_page_table(c, st);
}

int lckv_cache_lengths(const lckv_cache_t* c, int32_t* host_out, int32_t batch, void* stream)
{
    if (!c || !host_out || batch < 1 || batch > c->cfg.max_batch) return LCKV_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!cuda_ok(cudaMemcpyAsync(host_out, c->d_lens, (size_t)batch * 4, cudaMemcpyDeviceToHost, st)))
        return LCKV_ECUDA;
    return cuda_ok(cudaStreamSynchronize(st)) ? LCKV_OK : LCKV_ECUDA;
}

int lckv_cache_status(const lckv_cache_t* c, int32_t* host_status, void* stream)
{
    if (!c || !host_status) return LCKV_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!cuda_ok(cudaMemcpyAsync(host_status, c->d_status, 4, cudaMemcpyDeviceToHost, st)))
        return LCKV_ECUDA;
    return cuda_ok(cudaStreamSynchronize(st)) ? LCKV_OK : LCKV_ECUDA;
}

int lckv_cache_set_wait_limit(lckv_cache_t* c, uint32_t polls)
{
    if (!c) return LCKV_EINVAL;
    c->wait_limit = polls;
    drop_graph(c);   // a captured step carries the old limit in its kernel arguments
    return LCKV_OK;
}

int lckv_cache_set_worker_limit(lckv_cache_t* c, int32_t workers)
{
    if (!c || workers < 0 || workers > c->n_workers) return LCKV_EINVAL;
    c->active_workers = workers ? workers : c->n_workers;
    drop_graph(c);   // a captured step carries the old count in its kernel arguments
    return LCKV_OK;
}

int lckv_cache_slot_ptrs(const lckv_cache_t* c, int32_t slot, void** k, void** v)
{
    if (!c || !k || !v || slot < 0 || slot >= c->plan.n_slots) return LCKV_EINVAL;
    *k = slot_k(c, slot);
    *v = slot_v(c, slot);
    return LCKV_OK;
}

int lckv_cache_page_table(const lckv_cache_t* c, int32_t* host_out, int32_t* entries_per_seq)
{
    if (!c || !entries_per_seq || !c->cfg.page_rows) return LCKV_EINVAL;
    *entries_per_seq = c->pt_stride;
    if (host_out) std::memcpy(host_out, c->h_pt.data(), c->h_pt.size() * 4);
    return LCKV_OK;
}

int lckv_append_kv(lckv_cache_t* c, int32_t slot, const void* k_new, const void* v_new,
                   int32_t batch, int32_t advance_len, void* stream)
{
    if (!c || !k_new || !v_new || batch < 1 || batch > c->cfg.max_batch) return LCKV_EINVAL;
    if (slot < 0 || slot >= c->plan.n_slots) return LCKV_EINVAL;
    if (max_len(c, batch) + 1 > c->cfg.max_seq) return LCKV_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (int rc = ensure_pages(c, batch, 1)) return rc;
    if (int rc = sync_page_table(c, st)) return rc;
    if (int rc = launch_append(c, slot, k_new, v_new, batch, st)) return rc;
    if (advance_len) {
        if (int rc = launch_advance(c, batch, st)) return rc;
        mirror_advance(c, batch);
    }
    return LCKV_OK;
}

namespace {

// Tensor map of a row-major bf16 matrix [rows, cols] with boxes of box_rows x 64 columns; kept per
// (address, shape, box) so that repeated calls with the same weights do not re-encode.
int operand_map(lckv_cache* c, const void* ptr, uint64_t rows, uint64_t cols, int box_rows,
                CUtensorMap* out)
{
    for (const auto& m : c->operand_maps)
        if (m.ptr == ptr && m.rows == rows && m.cols == cols && m.box_rows == box_rows) {
            *out = m.tm;
            return LCKV_OK;
        }
    if (c->operand_maps.size() >= 256) c->operand_maps.clear();
    lckv_cache::OperandMap m;
    m.ptr = ptr; m.rows = rows; m.cols = cols; m.box_rows = box_rows;
    if (int rc = make_tensor_map_pitch(&m.tm, const_cast<void*>(ptr), rows, cols, cols * 2, box_rows))
        return rc;
    c->operand_maps.push_back(m);
    *out = m.tm;
    return LCKV_OK;
}

}  // namespace

int lckv_project_append_kv(lckv_cache_t* c, int32_t slot, const void* x, int32_t d_model,
                           const void* w_k, const void* w_v, const float* rope_cos,
                           const float* rope_sin, int32_t rope_positions, int32_t batch,
                           int32_t advance_len, void* stream)
{
    if (!c || !x || !w_k || !w_v || batch < 1 || batch > c->cfg.max_batch) return LCKV_EINVAL;
    if (slot < 0 || slot >= c->plan.n_slots) return LCKV_EINVAL;
    const int D = c->cfg.head_dim, F = c->cfg.n_kv_heads * D;
    if (d_model < 64 || d_model % 64 || F % lckv::kProjBM) return LCKV_EINVAL;
    if (((uintptr_t)x | (uintptr_t)w_k | (uintptr_t)w_v) & 15) return LCKV_EINVAL;
    if ((rope_cos == nullptr) != (rope_sin == nullptr)) return LCKV_EINVAL;
    if (((uintptr_t)rope_cos | (uintptr_t)rope_sin) & 15) return LCKV_EINVAL;
    if (rope_cos && (rope_positions < 1 || max_len(c, batch) >= rope_positions)) return LCKV_EINVAL;
    if (max_len(c, batch) + 1 > c->cfg.max_seq) return LCKV_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (int rc = ensure_pages(c, batch, 1)) return rc;
    if (int rc = sync_page_table(c, st)) return rc;

    // batch tile = N of the MMA: any multiple of 16 up to 256; equal tiles when the batch needs several
    const int n_btiles = (batch + 255) / 256;
    const int NB = ((batch + n_btiles - 1) / n_btiles + 15) / 16 * 16;
    // k-step width: a weight row is fetched in runs of 128 * k_boxes bytes.  Runs of 256 bytes are
    // served better by the memory than runs of 128 (fewer row activations per byte: 17.1 -> 15.2 us
    // per call at the 7B width, B = 16); used while at least three stages still fit.
    const int smem_budget = 222 * 1024;
    const int k_boxes = (d_model % 128 == 0 && smem_budget / lckv::proj_stage_bytes(NB, 2) >= 3) ? 2 : 1;
    // Stages: as many as fit beside a second CTA on the SM (so that the start of one call overlaps the
    // tail of the kernel before it) if that leaves at least four; else as many as fit alone.
    const int stage_bytes = lckv::proj_stage_bytes(NB, k_boxes);
    int n_stages = (111 * 1024) / stage_bytes;
    if (n_stages < 4) n_stages = smem_budget / stage_bytes;
    if (n_stages > 8) n_stages = 8;
    if (n_stages < 2) return LCKV_EINVAL;
    CUtensorMap tx, tk, tv;
    if (int rc = operand_map(c, x, (uint64_t)batch, (uint64_t)d_model, NB, &tx)) return rc;
    if (int rc = operand_map(c, w_k, (uint64_t)F, (uint64_t)d_model, lckv::kProjBM, &tk)) return rc;
    if (int rc = operand_map(c, w_v, (uint64_t)F, (uint64_t)d_model, lckv::kProjBM, &tv)) return rc;

    lckv::ProjParams p;
    p.K = slot_k(c, slot);
    p.V = slot_v(c, slot);
    p.lens = c->d_lens;
    p.rope_cos = rope_cos;
    p.rope_sin = rope_sin;
    p.status = c->d_status;
    p.page_table = c->d_pt;
    p.T_cap = c->cfg.max_seq;
    p.pt_stride = c->pt_stride;
    p.page_shift = c->page_shift;
    p.B = batch;
    p.H_kv = c->cfg.n_kv_heads;
    p.D = D;
    p.d_model = d_model;
    p.NB = NB;
    p.n_stages = n_stages;
    p.n_sink = c->cfg.stream_sink;
    p.k_tiles = F / lckv::kProjBM;
    p.rope_positions = rope_positions;
    // Few feature tiles (small batch): split d_model over a cluster so that more SMs stream weights.
    const int tiles = 2 * p.k_tiles * ((batch + NB - 1) / NB);
    const int n_k = d_model / (lckv::kProjBoxCols * k_boxes);
    p.k_boxes = k_boxes;
    int ks = 1;
    while (ks < 8 && tiles * ks * 2 <= c->sm_count && n_k % (ks * 2) == 0 && n_k / (ks * 2) >= 4) ks *= 2;
    p.k_split = ks;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(2 * p.k_tiles, (batch + NB - 1) / NB, ks);
    lc.blockDim = dim3(lckv::kProjThreads);
    lc.dynamicSmemBytes = lckv::proj_smem_bytes(NB, n_stages, k_boxes);
    lc.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 1;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = ks;
    // the kernel orders itself after its predecessor with griddepcontrol.wait (weights first)
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at;
    lc.numAttrs = 2;
    if (!cuda_ok(cudaLaunchKernelEx(&lc, lckv::project_kv_kernel, p, tx, tk, tv))) return LCKV_ECUDA;
    if (advance_len) {
        if (int rc = launch_advance(c, batch, st)) return rc;
        mirror_advance(c, batch);
    }
    return LCKV_OK;
}

int lckv_decode_attention(lckv_cache_t* c, int32_t slot, int32_t mode, const void* q, void* out,
                          float* lse, int32_t batch, void* stream)
{
    if (!c || !q || !out || batch < 1 || batch > c->cfg.max_batch) return LCKV_EINVAL;
    if (slot < 0 || slot >= c->plan.n_slots) return LCKV_EINVAL;
    if (mode != LCKV_MODE_CONDENSED && mode != LCKV_MODE_STANDARD) return LCKV_EINVAL;
    if (max_len(c, batch) + mode > c->cfg.max_seq) return LCKV_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (int rc = ensure_pages(c, batch, mode)) return rc;
    if (int rc = sync_page_table(c, st)) return rc;
    if (int rc = launch_plan(c, batch, st)) return rc;
    return launch_attention(c, slot, mode, q, out, lse, batch, st);
}

int lckv_layer_stack_step(lckv_cache_t* c, const void* const* q_layers, void* const* out_layers,
                          const void* const* k_new_layers, const void* const* v_new_layers,
                          int32_t batch, void* stream)
{
    if (!c || !q_layers || !out_layers || !k_new_layers || !v_new_layers) return LCKV_EINVAL;
    if (batch < 1 || batch > c->cfg.max_batch) return LCKV_EINVAL;
    const int L = c->cfg.n_layers;
    for (int l = 0; l < L; ++l) {
        if (!q_layers[l] || !out_layers[l]) return LCKV_EINVAL;
        if (c->plan.write_slot[l] >= 0 && (!k_new_layers[l] || !v_new_layers[l])) return LCKV_EINVAL;
    }
    if (max_len(c, batch) + 1 > c->cfg.max_seq) return LCKV_ECAPACITY;
    return run_step(c, q_layers, out_layers, k_new_layers, v_new_layers, batch,
                    static_cast<cudaStream_t>(stream));
}

int lckv_layer_stack_step_host(lckv_cache_t* c, const void* const* q_host, void* const* out_host,
                               const void* const* kn_host, const void* const* vn_host,
                               int32_t batch, void* stream)
{
    if (!c || !q_host || !out_host || !kn_host || !vn_host) return LCKV_EINVAL;
    if (!c->cfg.host_staging) return LCKV_EINVAL;
    if (batch < 1 || batch > c->cfg.max_batch) return LCKV_EINVAL;
    const int L = c->cfg.n_layers;
    for (int l = 0; l < L; ++l) {
        if (!q_host[l] || !out_host[l]) return LCKV_EINVAL;
        if (c->plan.write_slot[l] >= 0 && (!kn_host[l] || !vn_host[l])) return LCKV_EINVAL;
    }
    if (max_len(c, batch) + 1 > c->cfg.max_seq) return LCKV_ECAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t q_bytes = (size_t)batch * c->cfg.n_q_heads * c->cfg.head_dim * 2;
    const size_t o_bytes = (size_t)batch * c->cfg.n_q_heads * c->cfg.head_dim * (c->cfg.out_dtype ? 4 : 2);
    const size_t kv_bytes = (size_t)batch * c->cfg.n_kv_heads * c->cfg.head_dim * 2;
    std::vector<const void*> dq(L), dk(L, nullptr), dv(L, nullptr);
    std::vector<void*> dout(L);
    std::vector<const void*> hk, hv;
    int kv_i = 0;
    for (int l = 0; l < L; ++l) {
        dq[l] = c->base + c->lay.off_stage_q + (size_t)l * c->lay.stage_q_bytes;
        dout[l] = c->base + c->lay.off_stage_out + (size_t)l * c->lay.stage_out_bytes;
        if (c->plan.write_slot[l] >= 0) {
            uint8_t* sk = c->base + c->lay.off_stage_kv + (size_t)(2 * kv_i) * c->lay.stage_kv_bytes;
            dk[l] = sk;
            dv[l] = sk + c->lay.stage_kv_bytes;
            hk.push_back(kn_host[l]);
            hv.push_back(vn_host[l]);
            ++kv_i;
        }
    }
    uint8_t* skv = c->base + c->lay.off_stage_kv;
    // Copies run on two streams of the cache's own, so that the inputs of later layers arrive and
    // the outputs of earlier layers leave while the layers in between compute.  The layers are cut
    // into chunks; a chunk starts once its queries are on the device, and its outputs are fetched
    // once it is done.  The caller's stream ends up waiting for the last copy.
    const int n_chunks = L < 8 ? L : 8;
    if (!c->s_in) {
        if (!cuda_ok(cudaStreamCreateWithFlags(&c->s_in, cudaStreamNonBlocking)) ||
            !cuda_ok(cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking)))
            return LCKV_ECUDA;
    }
    while ((int)c->ev.size() < 3 + 2 * n_chunks) {
        cudaEvent_t e;
        if (!cuda_ok(cudaEventCreateWithFlags(&e, cudaEventDisableTiming))) return LCKV_ECUDA;
        c->ev.push_back(e);
    }
    cudaEvent_t ev_start = c->ev[0], ev_kv = c->ev[1], ev_out = c->ev[2];
    // everything that can refuse the step comes before the first copy is queued
    if (int rc = ensure_pages(c, batch, 1)) return rc;
    if (int rc = sync_page_table(c, st)) return rc;
    // staging buffers are free once everything queued on the caller's stream so far has run
    if (!cuda_ok(cudaEventRecord(ev_start, st)) || !cuda_ok(cudaStreamWaitEvent(c->s_in, ev_start, 0)))
        return LCKV_ECUDA;
    if (int rc = copy_layers(skv, 2 * c->lay.stage_kv_bytes, hk.data(), (int)hk.size(), kv_bytes, true, c->s_in))
        return rc;
    if (int rc = copy_layers(skv + c->lay.stage_kv_bytes, 2 * c->lay.stage_kv_bytes, hv.data(),
                             (int)hv.size(), kv_bytes, true, c->s_in))
        return rc;
    if (!cuda_ok(cudaEventRecord(ev_kv, c->s_in)) || !cuda_ok(cudaStreamWaitEvent(st, ev_kv, 0)))
        return LCKV_ECUDA;
    StepHooks hooks;
    hooks.wait_before.assign(L, nullptr);
    hooks.record_after.assign(L, nullptr);
    std::vector<int> first(n_chunks + 1);
    for (int k = 0; k <= n_chunks; ++k) first[k] = (int)((int64_t)k * L / n_chunks);
    for (int k = 0; k < n_chunks; ++k) {
        const int l0 = first[k], n = first[k + 1] - l0;
        if (int rc = copy_layers(c->base + c->lay.off_stage_q + (size_t)l0 * c->lay.stage_q_bytes,
                                 c->lay.stage_q_bytes, q_host + l0, n, q_bytes, true, c->s_in))
            return rc;
        if (!cuda_ok(cudaEventRecord(c->ev[3 + 2 * k], c->s_in))) return LCKV_ECUDA;
        hooks.wait_before[l0] = c->ev[3 + 2 * k];
        hooks.record_after[l0 + n - 1] = c->ev[4 + 2 * k];
    }
    if (int rc = enqueue_step(c, dq.data(), dout.data(), dk.data(), dv.data(), batch, st, &hooks)) return rc;
    mirror_advance(c, batch);
    for (int k = 0; k < n_chunks; ++k) {
        const int l0 = first[k], n = first[k + 1] - l0;
        if (!cuda_ok(cudaStreamWaitEvent(c->s_out, c->ev[4 + 2 * k], 0))) return LCKV_ECUDA;
        if (int rc = copy_layers(c->base + c->lay.off_stage_out + (size_t)l0 * c->lay.stage_out_bytes,
                                 c->lay.stage_out_bytes, const_cast<const void* const*>(out_host) + l0, n,
                                 o_bytes, false, c->s_out))
            return rc;
    }
    if (!cuda_ok(cudaEventRecord(ev_out, c->s_out)) || !cuda_ok(cudaStreamWaitEvent(st, ev_out, 0)))
        return LCKV_ECUDA;
    return LCKV_OK;
}

int lckv_prefill_write_kv(lckv_cache_t* c, int32_t slot, const void* k, const void* v,
                          int32_t n_max, int32_t batch, void* stream)
{
    if (!c || !k || !v || slot < 0 || slot >= c->plan.n_slots) return LCKV_EINVAL;
    if (int rc = prefill_check(c, n_max, batch, false)) return rc;
    if (int rc = sync_page_table(c, static_cast<cudaStream_t>(stream))) return rc;
    return launch_prefill_write(c, slot, k, v, n_max, batch, static_cast<cudaStream_t>(stream));
}

int lckv_prefill_attention(lckv_cache_t* c, int32_t slot, int32_t mode, const void* q, void* out,
                           int32_t n_max, int32_t batch, void* stream)
{
    if (!c || !q || !out || slot < 0 || slot >= c->plan.n_slots) return LCKV_EINVAL;
    if (mode != LCKV_MODE_CONDENSED && mode != LCKV_MODE_STANDARD) return LCKV_EINVAL;
    if (int rc = prefill_check(c, n_max, batch, true)) return rc;
    if (int rc = sync_page_table(c, static_cast<cudaStream_t>(stream))) return rc;
    return launch_prefill_attention(c, slot, mode, q, out, n_max, batch,
                                    static_cast<cudaStream_t>(stream));
}

int lckv_prefill_iteration(lckv_cache_t* c, const void* const* q_layers, void* const* out_layers,
                           const void* const* k_layers, const void* const* v_layers, int32_t n_max,
                           int32_t batch, void* stream)
{
    if (!c || !q_layers || !out_layers || !k_layers || !v_layers) return LCKV_EINVAL;
    if (int rc = prefill_check(c, n_max, batch, true)) return rc;
    const Plan& pl = c->plan;
    const int L = c->cfg.n_layers;
    for (int l = 0; l < L; ++l) {
        if (!q_layers[l] || !out_layers[l]) return LCKV_EINVAL;
        if (pl.write_slot[l] >= 0 && (!k_layers[l] || !v_layers[l])) return LCKV_EINVAL;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (int rc = sync_page_table(c, st)) return rc;
    for (int l = 0; l < L; ++l) {
        if (pl.write_slot[l] >= 0 && pl.write_before[l])
            if (int rc = launch_prefill_write(c, pl.write_slot[l], k_layers[l], v_layers[l], n_max, batch, st))
                return rc;
        if (int rc = launch_prefill_attention(c, pl.read_slot[l], pl.mode[l], q_layers[l],
                                              out_layers[l], n_max, batch, st))
            return rc;
    }
    for (int l = 0; l < L; ++l)
        if (pl.write_slot[l] >= 0 && !pl.write_before[l])
            if (int rc = launch_prefill_write(c, pl.write_slot[l], k_layers[l], v_layers[l], n_max, batch, st))
                return rc;
    return LCKV_OK;
}

int lckv_read_stream_probe(const void* src, size_t bytes, int32_t kind, int32_t repeats, float l2_keep,
                           uint32_t* dev_sum, int32_t* dev_status, void* stream)
{
    if (!src || !dev_sum || !dev_status || bytes < 16 || repeats < 1) return LCKV_EINVAL;
    if (!(l2_keep >= 0.f && l2_keep <= 1.f)) return LCKV_EINVAL;
    if (((uintptr_t)src & 15) || ((uintptr_t)dev_sum & 3) || ((uintptr_t)dev_status & 3)) return LCKV_EINVAL;
    if (kind < 0 || kind > 2 || (kind == 2 && ((uintptr_t)src & 31))) return LCKV_EINVAL;
    int sm = 0;
    if (int rc = device_sm_count(&sm)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (kind == 0) {
        // 8 resident blocks of 256 threads per SM: 16 KB of loads in flight per SM and loop trip
        lckv::read_stream_ldg_kernel<<<sm * 8, lckv::kProbeThreads, 0, st>>>(
            static_cast<const uint4*>(src), (uint64_t)(bytes / 16), dev_sum, repeats);
    } else if (kind == 2) {
        lckv::read_stream_ldg32_kernel<<<sm * 8, lckv::kProbeThreads, 0, st>>>(
            static_cast<const uint8_t*>(src), (uint64_t)(bytes / 32), dev_sum, repeats);
    } else {
        static std::once_flag once[64];
        int dev = 0;
        if (!cuda_ok(cudaGetDevice(&dev)) || dev < 0 || dev >= 64) return LCKV_ECUDA;
        bool ok = true;
        std::call_once(once[dev], [&] {
            ok = cuda_ok(cudaFuncSetAttribute(lckv::read_stream_bulk_kernel,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              lckv::kProbeSmemBytes));
        });
        if (!ok) return LCKV_ECUDA;
        lckv::read_stream_bulk_kernel<<<sm, lckv::kProbeThreads, lckv::kProbeSmemBytes, st>>>(
            static_cast<const uint8_t*>(src), (uint64_t)(bytes / lckv::kProbePiece), dev_sum, dev_status, repeats,
            l2_keep);
    }
    return cuda_ok(cudaGetLastError()) ? LCKV_OK : LCKV_ECUDA;
}

const char* lckv_status_string(int s)
{
    switch (s) {
        case LCKV_OK: return "ok";
        case LCKV_EINVAL: return "invalid argument";
        case LCKV_ECAPACITY: return "sequence capacity exceeded";
        case LCKV_ENOMEM: return "device buffer too small or misaligned";
        case LCKV_ECUDA: return "CUDA call failed";
        case LCKV_ETIMEOUT: return "device-side wait timed out";
        case LCKV_ESTATICLIMIT: return "size exceeds the static scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

int lckv_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"

// =============================================================================================
// Decode attention for callers that cannot allocate: scratch in a fixed device array.
// =============================================================================================
namespace {

constexpr int kStaticMaxWorkers = LCKV_STATIC_MAX_SMS * 8;  // worker records the scratch holds
constexpr int kStaticPreStride = LCKV_STATIC_MAX_BATCH + 64;
constexpr size_t kStOffPre = 0;
constexpr size_t kStOffStart = kStOffPre + 2 * (size_t)kStaticPreStride * 4;
constexpr size_t kStOffCounters = kStOffStart + 2 * (size_t)kStaticMaxWorkers * sizeof(lckv::WorkerStart);
constexpr size_t kStOffStatus = kStOffCounters + (size_t)kStaticMaxWorkers * 4;
constexpr size_t kStOffPartials = kStOffStatus + 256;
constexpr size_t kStBytes = kStOffPartials + 2 * (size_t)kStaticMaxWorkers * (128 + 4) * 4;
static_assert(kStBytes <= LCKV_STATIC_SCRATCH_BYTES, "static scratch too small for its limits");
static_assert(kStOffStart % 256 == 0 && kStOffCounters % 256 == 0 && kStOffPartials % 256 == 0,
              "sections must stay 256-byte aligned");

// Work plan, tickets, status word and split-K partials of lckv_decode_attention_static.  In host
// code this name is only a handle for cudaGetSymbolAddress, never a pointer to pass to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[LCKV_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;                            // guards the per-device set-up below
std::atomic<unsigned char*> g_static_ptr[kMaxDevices];  // device address of the array, per device;
                                                      // published last, after g_static_sms
int g_static_sms[kMaxDevices];

// Once per device, with that device current: resolve the array's device address.  Called with
// g_static_mutex held.
int static_setup(int dev)
{
    void* ptr = nullptr;
    if (!cuda_ok(cudaGetSymbolAddress(&ptr, g_static_scratch))) return LCKV_ECUDA;
    if (!ptr) return LCKV_ECUDA;
    int sms = 0;
    if (!cuda_ok(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) return LCKV_ECUDA;
    if (!cuda_ok(cudaFuncSetAttribute(lckv::attn_alu_kernel<128>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      lckv::kAluSmemBytes)) ||
        !cuda_ok(cudaFuncSetAttribute(lckv::attn_alu_kernel<64>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      lckv::kAluSmemBytes)))
        return LCKV_ECUDA;
    g_static_sms[dev] = sms;
    g_static_ptr[dev].store(static_cast<unsigned char*>(ptr), std::memory_order_release);
    return LCKV_OK;
}

}  // namespace

extern "C" int lckv_decode_attention_static(const void* k, const void* v, const int32_t* lens,
                                            const void* q, void* out, float* lse,
                                            int32_t* dev_status, int32_t batch, int32_t n_q_heads,
                                            int32_t n_kv_heads, int32_t head_dim, int64_t max_seq,
                                            int32_t mode, float softmax_scale, int32_t out_dtype,
                                            void* stream)
{
    if (!k || !v || !lens || !q || !out) return LCKV_EINVAL;
    // k, v move by 16-byte bulk copies, q and out by 128-bit loads and stores: a pointer off that
    // grid would fault on the device, so it is refused here
    if (((uintptr_t)k | (uintptr_t)v | (uintptr_t)q | (uintptr_t)out) & 15) return LCKV_EINVAL;
    if (((uintptr_t)lens | (uintptr_t)lse | (uintptr_t)dev_status) & 3) return LCKV_EINVAL;
    if (batch < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads) return LCKV_EINVAL;
    if (head_dim != 64 && head_dim != 128) return LCKV_EINVAL;
    if (max_seq < 1 || max_seq > 0x7fffffff) return LCKV_EINVAL;
    if (mode != LCKV_MODE_CONDENSED && mode != LCKV_MODE_STANDARD) return LCKV_EINVAL;
    if (out_dtype != 0 && out_dtype != 1) return LCKV_EINVAL;
    if (!(softmax_scale >= 0.f) || !std::isfinite(softmax_scale)) return LCKV_EINVAL;
    if (batch > LCKV_STATIC_MAX_BATCH) return LCKV_ESTATICLIMIT;
    if ((uint64_t)batch * (((uint64_t)max_seq + 15) / 16) >= (1ull << 31)) return LCKV_EINVAL;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return LCKV_ECUDA;
    if (dev < 0 || dev >= kMaxDevices) return LCKV_ESTATICLIMIT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* base = g_static_ptr[dev].load(std::memory_order_acquire);
    if (!base) {
        // The set-up calls are not stream work and must not land in a capture.
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (!cuda_ok(cudaStreamIsCapturing(st, &cs))) return LCKV_ECUDA;
        if (cs != cudaStreamCaptureStatusNone) return LCKV_EINVAL;
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev].load(std::memory_order_acquire))
            if (int rc = static_setup(dev)) return rc;
        base = g_static_ptr[dev].load(std::memory_order_acquire);
    }
    const int sms = g_static_sms[dev];
    const int n_workers = sms * lckv::kAluWarps * lckv::kAluCtas;
    if (sms > LCKV_STATIC_MAX_SMS || n_workers > kStaticMaxWorkers) return LCKV_ESTATICLIMIT;
    uint32_t* d_pre = reinterpret_cast<uint32_t*>(base + kStOffPre);
    lckv::WorkerStart* d_start = reinterpret_cast<lckv::WorkerStart*>(base + kStOffStart);
    int32_t* d_counters = reinterpret_cast<int32_t*>(base + kStOffCounters);
    int32_t* d_status = dev_status ? dev_status : reinterpret_cast<int32_t*>(base + kStOffStatus);

    // The array keeps whatever the previous call left: the tickets must start at zero.
    if (!cuda_ok(cudaMemsetAsync(d_counters, 0, (size_t)n_workers * 4, st))) return LCKV_ECUDA;
    if (!cuda_ok(cudaMemsetAsync(d_status, 0, 4, st))) return LCKV_ECUDA;

    const int R = lckv::kAluSlotBytes / (head_dim * 2);
    lckv::plan_kernel<<<1, 1024, 0, st>>>(lens, batch, R, n_q_heads, n_workers, d_pre,
                                          kStaticPreStride, d_start, (int)max_seq);
    if (!cuda_ok(cudaGetLastError())) return LCKV_ECUDA;

    lckv::AttnParams p;
    p.K = static_cast<const uint16_t*>(k);
    p.V = static_cast<const uint16_t*>(v);
    p.q = static_cast<const uint16_t*>(q);
    p.out = out;
    p.lse = lse;
    p.lens = lens;
    p.pre = d_pre + (size_t)mode * kStaticPreStride;
    p.start = d_start + (size_t)mode * n_workers;
    p.partials = reinterpret_cast<float*>(base + kStOffPartials);
    p.counters = d_counters;
    p.counters2 = nullptr;
    p.status = d_status;
    p.T_cap = max_seq;
    p.B = batch;
    p.H_q = n_q_heads;
    p.H_kv = n_kv_heads;
    p.mode = mode;
    p.n_workers = n_workers;
    p.out_f32 = out_dtype;
    p.early_kv = 0;
    p.wait_limit = lckv::kDefaultWaitLimit;
    p.l2_keep = 0.f;
    p.page_table = nullptr;
    p.pt_stride = 0;
    p.page_shift = 0;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / std::sqrt((float)head_dim);
    p.scale_log2 = scale * 1.4426950408889634f;
    if (head_dim == 128)
        lckv::attn_alu_kernel<128><<<sms * lckv::kAluCtas, lckv::kAluWarps * 32, lckv::kAluSmemBytes, st>>>(p);
    else
        lckv::attn_alu_kernel<64><<<sms * lckv::kAluCtas, lckv::kAluWarps * 32, lckv::kAluSmemBytes, st>>>(p);
    return cuda_ok(cudaGetLastError()) ? LCKV_OK : LCKV_ECUDA;
}
