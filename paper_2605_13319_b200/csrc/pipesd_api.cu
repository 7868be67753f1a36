// Host engine and C ABI of the NAV verify library: context, paged-KV bookkeeping, launch plan.
// Every step of the pass runs in the kernels of this directory; the host only validates, keeps the
// page tables and request lengths, uploads the per-call metadata and launches.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <cmath>
#include <deque>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/pipesd.h"
#include "attention.cuh"
#include "common.cuh"
#include "gemm.cuh"
#include "gemm_dense.cuh"
#include "layers.cuh"
#include "reject.cuh"

using namespace pipesd;

namespace {

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

struct Request {
    bool open = false;
    int len = 0;        // committed positions
    int tentative = 0;  // rows written by a verify that has not been committed yet (k+1), else 0
    int spec = 0;       // rows written by commit-on-device verifies still in flight (each planned as if its predecessors
                        // had accepted every draft); the host learns the committed length at the next pipesd_ctx_sync
    int pending = -1;   // recorded pending token (pipesd_kv_rollback with next_token, or a commit on device), -1: none
    std::vector<int> pages;
};

struct GemmW {
    uint4* packed = nullptr;     // MMA-fragment order (small-M kernel)
    uint4* packed_u = nullptr;   // tensor-core operand order (dense kernel; only when max_rows > 32)
    int N = 0, K = 0;
};

struct LayerW {
    GemmW qkv, o, gu, dn;
    float *n1 = nullptr, *n2 = nullptr;
};

// Fixed offsets of the per-call metadata block (same layout in pinned host staging and on device).
struct MetaLayout {
    size_t row_item, row_pos, row_tok, it_slot, it_row0, it_rows, it_base, it_nsplit, it_chunk, it_part0, it_order, u, rej, total;
};

MetaLayout meta_layout(int max_rows, int max_items) {
    MetaLayout m;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 16); return r; };
    m.row_item = take(4 * (size_t)max_rows);
    m.row_pos = take(4 * (size_t)max_rows);
    m.row_tok = take(4 * (size_t)max_rows);
    m.it_slot = take(4 * (size_t)max_items);
    m.it_row0 = take(4 * (size_t)max_items);
    m.it_rows = take(4 * (size_t)max_items);
    m.it_base = take(4 * (size_t)max_items);
    m.it_nsplit = take(4 * (size_t)max_items);
    m.it_chunk = take(4 * (size_t)max_items);
    m.it_part0 = take(4 * (size_t)max_items);
    m.it_order = take(4 * (size_t)max_items);
    m.u = take(4 * (size_t)max_rows);
    m.rej = take(sizeof(RejectItem) * (size_t)max_items);
    m.total = align_up(o);
    return m;
}

struct Derived {
    int Nqkv, qd, kvd, max_pages, max_items;
    size_t part_floats;  // floats in each of the two KV staging arrays
};

Derived derive(const pipesd_model_cfg& c) {
    Derived d;
    d.qd = c.n_q_heads * c.head_dim;
    d.kvd = c.n_kv_heads * c.head_dim;
    d.Nqkv = d.qd + 2 * d.kvd;
    // block-table rows are read four entries at a time (one 64-key tile of 16-position pages): padded to a
    // multiple of four entries with one spare group
    d.max_pages = ((c.max_seq + c.page_size - 1) / c.page_size + 3) / 4 * 4 + 4;
    d.max_items = std::min(c.max_requests, c.max_rows);
    // two staging arrays for pipesd_debug_read_kv / write_kv: 256 positions of K and of V per round
    size_t best = (size_t)256 * d.kvd / 2 + 64;
    d.part_floats = best;
    return d;
}

struct WsLayout {
    size_t x, xf_h, qbuf, xf_attn, xf_act, logits, partA, partB, ssqA, ssqB, o_part, m_part, l_part, tickets, cs, sn, kvoff, stats, results, meta,
        block_tab, qstage, req_state, never_flag, total;
};

WsLayout ws_layout(const pipesd_model_cfg& c, const Derived& d) {
    WsLayout w;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes); return r; };
    const size_t M = c.max_rows;
    w.x = take(4 * M * c.d_model);
    // split-bf16 activation arrays: 4 bytes per element, token count padded to whole token blocks (of up to 160 tokens
    // plus rounding in the dense kernel's layout)
    w.xf_h = take(4 * (M + 176) * c.d_model);
    w.qbuf = take(4 * M * d.qd);
    w.xf_attn = take(4 * (M + 176) * d.qd);
    w.xf_act = take(4 * (M + 176) * c.d_ffn);
    w.logits = take(4 * M * c.vocab);
    w.partA = take(4 * d.part_floats);
    w.partB = take(4 * d.part_floats);
    const size_t nssq = (c.d_model + 127) / 128;
    w.ssqA = take(4 * nssq * M);
    w.ssqB = take(4 * nssq * M);
    const size_t slots = M * c.n_q_heads * kAttnMaxSplits;               // one per (row, head, key split)
    w.o_part = take(4 * slots * c.head_dim);
    w.m_part = take(4 * slots);
    w.l_part = take(4 * slots);
    w.tickets = take(4 * M * c.n_q_heads);   // one per (item, KV head, row group); zero between launches
    w.cs = take(4 * M * (c.head_dim / 2));
    w.sn = take(4 * M * (c.head_dim / 2));
    w.kvoff = take(8 * M);
    w.stats = take(sizeof(RowStat) * M * kStatSplits);
    w.results = take(sizeof(RejectOut) * d.max_items + 16);   // + the device error word, read back with the results
    w.meta = take(meta_layout(c.max_rows, d.max_items).total);
    w.block_tab = take(4 * (size_t)c.max_requests * d.max_pages);
    w.qstage = take(4 * M * c.vocab);
    w.req_state = take(sizeof(ReqState) * (size_t)c.max_requests);
    w.never_flag = take(16);
    w.total = o;
    return w;
}

size_t packed_bytes(int N, int K) { return align_up(gemm_packed_bytes(N, K)); }

size_t weights_bytes(const pipesd_model_cfg& c, const Derived& d) {
    const size_t copies = c.max_rows > 32 ? 2 : 1;      // passes of more than 32 rows read the weights in another order
    size_t per_layer = copies * (packed_bytes(d.Nqkv, c.d_model) + packed_bytes(c.d_model, d.qd) +
                                 packed_bytes(2 * c.d_ffn, c.d_model) + packed_bytes(c.d_model, c.d_ffn)) +
                       2 * align_up(4 * (size_t)c.d_model);
    return (size_t)c.n_layers * per_layer + align_up((size_t)c.vocab * c.d_model * 2) +
           copies * packed_bytes(c.vocab, c.d_model) + align_up(4 * (size_t)c.d_model);
}

size_t kv_bytes(const pipesd_model_cfg& c) {
    return (size_t)c.n_layers * c.n_pages * 2 * c.n_kv_heads * c.page_size * c.head_dim * 2;
}

// Kernel attributes (shared-memory limits, cluster sizes) belong to a device: set once per device ordinal, with that
// device current, whichever entry point gets there first.
constexpr int kMaxDevices = 64;
std::mutex g_dev_mu;
bool g_dev_ready[kMaxDevices] = {false};

cudaError_t init_attrs_current_device() {
    cudaError_t e;
    if ((e = gemm_init_attrs()) != cudaSuccess) return e;
    const void* dense_fns[4] = {(const void*)gemm_dense_kernel<kPlain>, (const void*)gemm_dense_kernel<kQkvRope>,
                                (const void*)gemm_dense_kernel<kResid>, (const void*)gemm_dense_kernel<kSwiglu>};
    for (const void* fn : dense_fns) {
        if ((e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kDenseSmemWhole)) != cudaSuccess) return e;
        if ((e = cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, 100)) != cudaSuccess) return e;
    }
    e = cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_smem_bytes(128, kAttnMaxRows, false));
    if (e != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout, 100)) != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_smem_bytes(64, kAttnMaxRows, false));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
}

int ensure_device_ready() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PIPESD_E_CUDA;
    std::lock_guard<std::mutex> lock(g_dev_mu);
    if (!g_dev_ready[dev]) {
        if (init_attrs_current_device() != cudaSuccess) return PIPESD_E_CUDA;
        g_dev_ready[dev] = true;
    }
    return PIPESD_OK;
}

int check_cfg(const pipesd_model_cfg* c) {
    if (!c) return PIPESD_E_INVALID;
    if (c->n_layers < 1 || c->d_model < 16 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->d_ffn < 16 ||
        c->vocab < 16)
        return PIPESD_E_INVALID;
    if (c->head_dim != 64 && c->head_dim != 128) return PIPESD_E_INVALID;
    if (c->d_model % 16 || c->d_ffn % 16 || c->vocab % 16 || c->d_model > 8192) return PIPESD_E_INVALID;
    if (c->n_q_heads % c->n_kv_heads) return PIPESD_E_INVALID;
    if (c->page_size < 8 || c->page_size > 256 || c->page_size % 8 || c->n_pages < 1 || c->max_requests < 1)
        return PIPESD_E_INVALID;
    if (c->max_draft < 1 || c->max_draft > kMaxItemRows - 1) return PIPESD_E_INVALID;
    if (c->max_rows < c->max_draft + 1 || c->max_rows > 4096 || c->max_seq < 1) return PIPESD_E_INVALID;
    if (!(c->rms_eps >= 0.f) || !(c->rope_base > 1.f)) return PIPESD_E_INVALID;
    if (c->reserved != 0) return PIPESD_E_INVALID;
    return PIPESD_OK;
}

// Copy rows of one layer between a contiguous [n_pos][Hkv*hd] bf16 staging array and the pages.
__global__ void kv_copy_kernel(uint16_t* __restrict__ kv_pool, uint16_t* __restrict__ stage_k,
                               uint16_t* __restrict__ stage_v, const int32_t* __restrict__ bt, int pos0, int n_pos,
                               int layer, int n_pages, int page_size, int Hkv, int hd, int to_pool) {
    const int w = Hkv * hd;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)n_pos * w;
         i += (size_t)gridDim.x * blockDim.x) {
        int p = (int)(i / w), c = (int)(i % w), head = c / hd, e = c % hd;
        int pos = pos0 + p, page = bt[pos / page_size], slot = pos % page_size;
        size_t ko = kv_index(layer, n_pages, page, 0, Hkv, head, page_size, slot, hd, e);
        size_t vo = kv_index(layer, n_pages, page, 1, Hkv, head, page_size, slot, hd, e);
        if (to_pool) { kv_pool[ko] = stage_k[i]; kv_pool[vo] = stage_v[i]; }
        else { stage_k[i] = kv_pool[ko]; stage_v[i] = kv_pool[vo]; }
    }
}

}  // namespace

struct pipesd_ctx {
    pipesd_model_cfg cfg;
    Derived dv;
    WsLayout ws;
    MetaLayout ml;
    cudaStream_t st = nullptr;
    // device
    uint16_t* emb = nullptr;
    GemmW lm;
    float* final_norm = nullptr;
    std::vector<LayerW> layers;
    uint16_t* kv_pool = nullptr;
    char* wsp = nullptr;
    // host
    std::vector<Request> reqs;
    std::vector<int> free_pages;
    static constexpr int kStages = 4;
    char* h_meta[kStages] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t ev_meta[kStages] = {nullptr, nullptr, nullptr, nullptr};
    int stage = 0;
    // Calls whose results (and device error word) have been copied towards the host but not looked at yet, oldest
    // first; at most kStages of them (one pinned staging buffer each).
    struct InflightItem { int slot, k, commit; };
    struct Inflight {
        pipesd_verify_result* dst = nullptr;   // caller's array (null: a prefill or a self-test, only the error word matters)
        std::vector<InflightItem> items;
        int buf = 0;                           // staging buffer
    };
    RejectOut* h_results[kStages] = {nullptr, nullptr, nullptr, nullptr};
    std::deque<Inflight> inflight;
    int res_buf = 0;
    int last_rows = 0;
    int attn_slots[kAttnMaxRows / 16 + 1][2] = {};   // [query rows / 16][cut-down third ring slot]: CTAs of the attention
                                                     // kernel the device keeps resident at once
    int n_sm = 148;             // SMs of the context's device
    bool force_dense = false;   // harness switch: the dense kernels also for passes of at most 32 rows
    bool pass_dense = false;    // the pass being enqueued runs on the dense kernels
    // bytes of the O and gate/up weights the attention kernel pulls into L2 once its K/V has landed (measured: all of O
    // and 16 MB of gate/up; more gains nothing, an SM takes data in only about 1.4 times faster than HBM delivers it)
    size_t pf_attn[2] = {(size_t)64 << 20, (size_t)16 << 20};
    uint32_t pf_depth = 32u << 10;   // bytes per successor CTA that a GEMM pulls into L2 for the next GEMM
    std::string err;
    // launch accounting
    int64_t n_launch = 0, n_gemm = 0;
    double gemm_bytes = 0.0;
    bool time_gemms = false;
    std::vector<cudaEvent_t> prof_ev;   // start/stop pairs
    size_t prof_used = 0;

    template <typename T>
    T* W(size_t off) const { return reinterpret_cast<T*>(wsp + off); }
    int* err_word() const { return reinterpret_cast<int*>(wsp + ws.results + sizeof(RejectOut) * dv.max_items); }
    PassMeta pass_meta() const {
        PassMeta m;
        const char* b = wsp + ws.meta;
        m.row_item = (const int32_t*)(b + ml.row_item);
        m.row_pos = (const int32_t*)(b + ml.row_pos);
        m.row_tok = (const int32_t*)(b + ml.row_tok);
        m.it_slot = (const int32_t*)(b + ml.it_slot);
        m.it_row0 = (const int32_t*)(b + ml.it_row0);
        m.it_rows = (const int32_t*)(b + ml.it_rows);
        m.it_base = (const int32_t*)(b + ml.it_base);
        m.it_nsplit = (const int32_t*)(b + ml.it_nsplit);
        m.it_chunk = (const int32_t*)(b + ml.it_chunk);
        m.it_part0 = (const int32_t*)(b + ml.it_part0);
        m.it_order = (const int32_t*)(b + ml.it_order);
        m.block_tab = W<int32_t>(ws.block_tab);
        m.max_pages = dv.max_pages;
        return m;
    }
};

namespace {

int fail(pipesd_ctx* c, int code, const char* what) {
    if (c) c->err = std::string(pipesd_strerror(code)) + ": " + what;
    return code;
}

int cuda_fail(pipesd_ctx* c, cudaError_t e, const char* where) {
    if (c) c->err = std::string("CUDA error at ") + where + ": " + cudaGetErrorString(e);
    return PIPESD_E_CUDA;
}

#define CU(call)                                                    \
    do {                                                            \
        cudaError_t e_ = (call);                                    \
        if (e_ != cudaSuccess) return cuda_fail(ctx, e_, #call);    \
    } while (0)

template <int MODE>
cudaError_t dense_launch_mode(const DenseArgs& da, dim3 grid, size_t smem, cudaStream_t st) {
    return launch_pdl(gemm_dense_kernel<MODE>, grid, dim3(kDenseThreads), smem, st, da);
}

// Launch one weight-streaming GEMM with accounting (and event timing when profiling is on).  next_N: output rows of
// the GEMM that consumes this one's activation output (0: none): its token-block plan fixes the layout written.
int launch_gemm(pipesd_ctx* ctx, int mode, const GemmW& w, GemmArgs a, int K, int next_N) {
    a.err = ctx->err_word();
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (ctx->time_gemms) {
        if (ctx->prof_used + 2 > ctx->prof_ev.size()) {
            for (int i = 0; i < 2; ++i) {
                cudaEvent_t e;
                CU(cudaEventCreate(&e));
                ctx->prof_ev.push_back(e);
            }
        }
        e0 = ctx->prof_ev[ctx->prof_used];
        e1 = ctx->prof_ev[ctx->prof_used + 1];
        ctx->prof_used += 2;
        CU(cudaEventRecord(e0, ctx->st));
    }
    if (ctx->pass_dense) {
        const XdPlan pin = dense_plan(a.M, a.N, ctx->n_sm);
        DenseArgs da = {};
        da.g = a;
        da.g.W = w.packed_u;
        da.g.KS = K / 16;
        const dim3 grid((a.N + 127) / 128, pin.n_tb);
        const DenseRing ring = dense_ring(pin.tbs, (int)(grid.x * grid.y), ctx->n_sm);
        da.g.stages = ring.stages;
        da.kc = ring.kc;
        da.g.pf = L2Prefetch{};
        da.tbs_in = pin.tbs;
        da.tbs_out = next_N > 0 ? dense_plan(a.M, next_N, ctx->n_sm).tbs : 0;
        const size_t smem = ring.smem;
        cudaError_t e;
        switch (mode) {
            case kQkvRope: e = dense_launch_mode<kQkvRope>(da, grid, smem, ctx->st); break;
            case kResid: e = dense_launch_mode<kResid>(da, grid, smem, ctx->st); break;
            case kSwiglu: e = dense_launch_mode<kSwiglu>(da, grid, smem, ctx->st); break;
            default: e = dense_launch_mode<kPlain>(da, grid, smem, ctx->st); break;
        }
        CU(e);
    } else {
        a.W = w.packed;
        const GemmPlan p = gemm_plan(a.M, a.N, K);
        CU(gemm_launch(mode, p, a, ctx->st));
    }
    if (e1) CU(cudaEventRecord(e1, ctx->st));
    ctx->n_launch += 1;
    ctx->n_gemm += 1;
    ctx->gemm_bytes += 2.0 * a.N * K + 4.0 * a.M * K + 4.0 * a.M * a.N;
    return PIPESD_OK;
}

struct ItemDesc {
    int slot, rows, mode, k;
    const int32_t* tokens;  // host, rows ids
    const float* q;         // device
    const float* u;         // host, k+1 (null when mode == 2)
    int base;               // cached positions the pass runs against
    int commit;             // kCommit*
    int tok0;               // id of the first row when tokens[0] asks for the recorded pending token
};

// Enqueue the copy of the result slots and the device error word into the next staging buffer and remember the call.
int push_inflight(pipesd_ctx* ctx, pipesd_verify_result* dst, std::vector<pipesd_ctx::InflightItem> items) {
    pipesd_ctx::Inflight f;
    f.dst = dst;
    f.items = std::move(items);
    f.buf = ctx->res_buf;
    ctx->res_buf = (ctx->res_buf + 1) % pipesd_ctx::kStages;
    CU(cudaMemcpyAsync(ctx->h_results[f.buf], ctx->W<RejectOut>(ctx->ws.results), sizeof(RejectOut) * ctx->dv.max_items + 4,
                       cudaMemcpyDeviceToHost, ctx->st));
    ctx->inflight.push_back(std::move(f));
    return PIPESD_OK;
}

// Make sure the request owns pages for `need_len` positions. All-or-nothing is checked by the caller.
int pages_needed(const pipesd_ctx* c, const Request& r, int need_len) {
    int need = (need_len + c->cfg.page_size - 1) / c->cfg.page_size;
    return std::max(0, need - (int)r.pages.size());
}

int grow_pages(pipesd_ctx* ctx, int slot, int need_len) {
    Request& r = ctx->reqs[slot];
    int add = pages_needed(ctx, r, need_len);
    if (add == 0) return PIPESD_OK;
    int first = (int)r.pages.size();
    for (int i = 0; i < add; ++i) {
        r.pages.push_back(ctx->free_pages.back());
        ctx->free_pages.pop_back();
    }
    int32_t* dst = ctx->W<int32_t>(ctx->ws.block_tab) + (size_t)slot * ctx->dv.max_pages + first;
    CU(cudaMemcpyAsync(dst, r.pages.data() + first, 4 * (size_t)add, cudaMemcpyHostToDevice, ctx->st));
    return PIPESD_OK;
}

void shrink_pages(pipesd_ctx* c, Request& r, int keep_len) {
    int keep = (keep_len + c->cfg.page_size - 1) / c->cfg.page_size;
    while ((int)r.pages.size() > keep) {
        c->free_pages.push_back(r.pages.back());
        r.pages.pop_back();
    }
}

// Upload the metadata of one pass and run the layer stack over M rows.
int run_pass(pipesd_ctx* ctx, const std::vector<ItemDesc>& items, bool want_logits, bool want_reject) {
    const pipesd_model_cfg& c = ctx->cfg;
    const Derived& dv = ctx->dv;
    const int n_items = (int)items.size();
    int M = 0;
    for (auto& it : items) M += it.rows;

    // ---- metadata
    const int sidx = ctx->stage;
    ctx->stage = (ctx->stage + 1) % pipesd_ctx::kStages;
    CU(cudaEventSynchronize(ctx->ev_meta[sidx]));
    char* hm = ctx->h_meta[sidx];
    const MetaLayout& ml = ctx->ml;
    auto I = [&](size_t off) { return reinterpret_cast<int32_t*>(hm + off); };
    float* hu = reinterpret_cast<float*>(hm + ml.u);
    RejectItem* hr = reinterpret_cast<RejectItem*>(hm + ml.rej);
    int row = 0, part0 = 0, max_nsplit = 1, u0 = 0;
    bool all_short = true;       // no split of the pass has more than two key tiles, the second a short one
    // attention work of the pass in (keys x CTA groups): a request gets the share of the device's resident CTAs that its
    // keys are of the pass's, so that the CTAs of the whole pass fill one wave
    // Rows per row group.  A CTA with up to 16 query rows shares its SM with a second one, a CTA with 17..32 does not;
    // in a pass whose largest request has 17..32 rows per KV head the groups are therefore cut at 16 (requests above 16
    // rows read their K/V twice) as long as that adds at most an eighth to the K/V the pass reads ...
    int rows_cap = kAttnMaxRows;
    {
        int maxR0 = 1;
        double keys = 0.0, keys16 = 0.0;
        for (int i = 0; i < n_items; ++i) {
            const int R_i = items[i].rows * (c.n_q_heads / c.n_kv_heads);
            maxR0 = std::max(maxR0, R_i);
            keys += (double)(items[i].base + items[i].rows);
            keys16 += (double)(items[i].base + items[i].rows) * ((R_i + 15) / 16);
        }
        // ... or at most a tenth to the bytes of the pass (weights once + K/V): a single request of 17 rows at the 7B shape
        const double kv_key = 4.0 * c.n_layers * c.n_kv_heads * c.head_dim;                     // K and V bytes of a position
        const double w_bytes = 2.0 * ((double)c.n_layers * ((double)(dv.Nqkv + dv.qd) * c.d_model + 3.0 * c.d_ffn * c.d_model) +
                                      (double)c.vocab * c.d_model);
        if (maxR0 > 16 && maxR0 <= 32 && (keys16 <= 1.125 * keys || (keys16 - keys) * kv_key <= 0.1 * (w_bytes + keys * kv_key)) &&
            ctx->attn_slots[1][0] > ctx->attn_slots[2][0])
            rows_cap = 16;
    }
    double pass_work = 0.0;
    for (int i = 0; i < n_items; ++i) {
        const int R_i = items[i].rows * (c.n_q_heads / c.n_kv_heads);
        pass_work += (double)(items[i].base + items[i].rows) * c.n_kv_heads * ((R_i + rows_cap - 1) / rows_cap);
    }
    {   // launch order of the attention CTAs: longest requests first
        int32_t* ord = I(ml.it_order);
        for (int i = 0; i < n_items; ++i) ord[i] = i;
        std::stable_sort(ord, ord + n_items, [&](int32_t x, int32_t y) {
            return items[x].base + items[x].rows > items[y].base + items[y].rows;
        });
    }
    for (int i = 0; i < n_items; ++i) {
        const ItemDesc& it = items[i];
        const int total = it.base + it.rows;
        const int R_i = it.rows * (c.n_q_heads / c.n_kv_heads);                  // query rows per KV head
        const int rg_i = (R_i + rows_cap - 1) / rows_cap;
        const int units_i = (int)std::min(1.0e9, std::ceil(pass_work / (double)total));
        const AttnSplit sp = attn_split_plan(total, c.page_size, std::max(units_i, c.n_kv_heads * rg_i),
                                             ctx->attn_slots[attn_rows_n(std::min(R_i, rows_cap)) / 16]);
        const int nsplit = sp.splits, chunk = sp.keys_per_split;
        if (chunk > kAttnTile + kAttnShortTail) all_short = false;
        I(ml.it_slot)[i] = it.slot;
        I(ml.it_row0)[i] = row;
        I(ml.it_rows)[i] = it.rows;
        I(ml.it_base)[i] = it.base;
        I(ml.it_nsplit)[i] = nsplit;
        I(ml.it_chunk)[i] = chunk;
        I(ml.it_part0)[i] = part0;
        max_nsplit = std::max(max_nsplit, nsplit);
        part0 += it.rows * c.n_q_heads * nsplit;
        hr[i].row0 = row;
        hr[i].k = it.k;
        hr[i].mode = it.mode;
        hr[i].u0 = u0;
        hr[i].q = it.q;
        hr[i].slot = it.slot;
        hr[i].base = it.base;
        hr[i].commit = it.commit;
        hr[i].reserved = 0;
        for (int j = 0; j < it.rows; ++j) {
            I(ml.row_item)[row + j] = i;
            I(ml.row_pos)[row + j] = it.base + j;
            I(ml.row_tok)[row + j] = j == 0 && it.tokens[0] < 0 ? it.tok0 : it.tokens[j];
        }
        for (int j = 0; j <= it.k; ++j) hu[u0 + j] = it.u ? it.u[j] : 0.f;
        u0 += it.k + 1;
        row += it.rows;
    }
    CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.meta, hm, ml.total, cudaMemcpyHostToDevice, ctx->st));
    CU(cudaEventRecord(ctx->ev_meta[sidx], ctx->st));

    // ---- layer stack
    const PassMeta meta = ctx->pass_meta();
    cudaStream_t st = ctx->st;
    float* x = ctx->W<float>(ctx->ws.x);
    uint32_t* xf_h = ctx->W<uint32_t>(ctx->ws.xf_h);
    float* qbuf = ctx->W<float>(ctx->ws.qbuf);
    uint32_t* xf_attn = ctx->W<uint32_t>(ctx->ws.xf_attn);
    uint32_t* xf_act = ctx->W<uint32_t>(ctx->ws.xf_act);
    float* ssqA = ctx->W<float>(ctx->ws.ssqA);   // sums of squares of the attention-norm (and final-norm) input
    float* ssqB = ctx->W<float>(ctx->ws.ssqB);   // ... of the FFN-norm input
    float* o_part = ctx->W<float>(ctx->ws.o_part);
    float* m_part = ctx->W<float>(ctx->ws.m_part);
    float* l_part = ctx->W<float>(ctx->ws.l_part);
    float* cs = ctx->W<float>(ctx->ws.cs);
    float* sn = ctx->W<float>(ctx->ws.sn);
    const int hd = c.head_dim, Hq = c.n_q_heads, Hkv = c.n_kv_heads, d = c.d_model, F = c.d_ffn;
    const int n_ssq = (d + 127) / 128;

    // Passes of more than 32 rows run their GEMMs on the dense kernels (every weight byte read once per block of up to 160
    // tokens); their activation arrays are in that kernel's operand order, with the token block size of the consumer.
    ctx->pass_dense = ctx->layers[0].qkv.packed_u != nullptr && (M > 32 || ctx->force_dense);
    const bool dense = ctx->pass_dense;
    const int tbs_qkv = dense ? dense_plan(M, dv.Nqkv, ctx->n_sm).tbs : 0, tbs_o = dense ? dense_plan(M, d, ctx->n_sm).tbs : 0;
    // Every kernel of the chain is launched with programmatic stream serialisation: it may start while its
    // predecessor drains and blocks in griddepcontrol.wait before touching the predecessor's output.
    {
        int n = M * hd / 2;
        CU(launch_pdl(rope_table_kernel, dim3((n + 127) / 128), dim3(128), 0, st, meta, M, hd, log((double)c.rope_base),
                      cs, sn, ctx->W<long long>(ctx->ws.kvoff), c.n_pages, Hkv, c.page_size));
        CU(launch_pdl(embed_kernel, dim3(M), dim3(kEmbedThreads), 0, st, x, (const uint16_t*)ctx->emb, meta.row_tok, M,
                      (const float*)ctx->layers[0].n1, d, xf_h, ssqA, n_ssq, tbs_qkv));
        ctx->n_launch += 2;
    }
    int max_item_rows = 1;
    for (auto& it : items) max_item_rows = std::max(max_item_rows, it.rows);
    const int maxR = max_item_rows * (Hq / Hkv);                      // query rows that share one KV head
    const int n_max = attn_rows_n(std::min(maxR, rows_cap));
    const int row_groups = (maxR + rows_cap - 1) / rows_cap;
    const size_t asmem = attn_smem_bytes(hd, n_max, all_short);
    GemmArgs base = {};
    base.M = M;
    base.eps = c.rms_eps;
    base.d_in = d;
    base.n_ssq = n_ssq;
    // depth of the L2 hints a kernel issues for its successor's weights (bytes per successor CTA)
    const uint32_t pf_depth = ctx->pf_depth;
    auto launch_attn = [&](int l) -> int {
        dim3 ag(max_nsplit, Hkv * row_groups, n_items);
        AttnArgs aa = {};
        aa.q = qbuf; aa.meta = meta; aa.kv_pool = ctx->kv_pool;
        aa.layer = l; aa.n_pages = c.n_pages; aa.page_size = c.page_size; aa.M = M; aa.Hq = Hq; aa.Hkv = Hkv;
        aa.rows_cap = rows_cap; aa.n_max = n_max; aa.slot_c = attn_slot_c_bytes(hd, all_short); aa.row_groups = row_groups;
        aa.o_part = o_part; aa.m_part = m_part; aa.l_part = l_part; aa.tickets = ctx->W<int>(ctx->ws.tickets);
        aa.xf_out = (uint16_t*)xf_attn; aa.xd_tbs = tbs_o; aa.err = ctx->err_word();
        if (!dense) {
            const LayerW& lw = ctx->layers[l];
            aa.pf_ptr[0] = reinterpret_cast<const unsigned char*>(lw.o.packed);
            aa.pf_len[0] = std::min(gemm_packed_bytes(d, dv.qd), ctx->pf_attn[0]);
            aa.pf_ptr[1] = reinterpret_cast<const unsigned char*>(lw.gu.packed);
            aa.pf_len[1] = std::min(gemm_packed_bytes(2 * F, d), ctx->pf_attn[1]);
        }
        if (hd == 128) CU(launch_pdl(attn_kernel<128>, ag, dim3(kAttnThreads), asmem, st, aa));
        else CU(launch_pdl(attn_kernel<64>, ag, dim3(kAttnThreads), asmem, st, aa));
        ctx->n_launch += 1;
        return PIPESD_OK;
    };
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerW& lw = ctx->layers[l];
        {   // q, k, v = W_qkv . norm(x); RoPE; K/V appended to the pages
            GemmArgs a = base;
            a.xf = (const uint4*)xf_h; a.N = dv.Nqkv; a.ssq_in = ssqA;
            a.q_out = qbuf; a.kv_pool = ctx->kv_pool; a.cs = cs; a.sn = sn;
            a.row_kvoff = ctx->W<long long>(ctx->ws.kvoff);
            a.Hq = Hq; a.Hkv = Hkv; a.hd = hd; a.layer = l; a.n_pages = c.n_pages; a.page_size = c.page_size;
            int rc_ = launch_gemm(ctx, kQkvRope, lw.qkv, a, d, 0);
            if (rc_) return rc_;
        }
        { int rc_ = launch_attn(l); if (rc_) return rc_; }
        {   // x += W_o . attn; xf_h = x * ffn gain; ssqB
            GemmArgs a = base;
            a.xf = (const uint4*)xf_attn; a.N = d; a.ssq_in = nullptr;
            a.x = x; a.xf_out = (uint16_t*)xf_h; a.gain_next = lw.n2; a.ssq_out = ssqB;
            a.pf = gemm_prefetch_of(lw.gu.packed, M, 2 * F, d, pf_depth);
            int rc_ = launch_gemm(ctx, kResid, lw.o, a, dv.qd, 2 * F);
            if (rc_) return rc_;
        }
        {   // act = silu(W_g . norm(x)) * (W_u . norm(x))
            GemmArgs a = base;
            a.xf = (const uint4*)xf_h; a.N = 2 * F; a.ssq_in = ssqB;
            a.xf_act = (uint16_t*)xf_act;
            a.pf = gemm_prefetch_of(lw.dn.packed, M, d, F, pf_depth);
            int rc_ = launch_gemm(ctx, kSwiglu, lw.gu, a, d, d);
            if (rc_) return rc_;
        }
        {   // x += W_d . act; xf_h = x * (next layer's attention gain | final gain); ssqA
            GemmArgs a = base;
            a.xf = (const uint4*)xf_act; a.N = d; a.ssq_in = nullptr;
            a.x = x; a.xf_out = (uint16_t*)xf_h;
            a.gain_next = l + 1 < c.n_layers ? ctx->layers[l + 1].n1 : ctx->final_norm;
            a.ssq_out = ssqA;
            if (l + 1 < c.n_layers) a.pf = gemm_prefetch_of(ctx->layers[l + 1].qkv.packed, M, dv.Nqkv, d, pf_depth);
            else if (want_logits) a.pf = gemm_prefetch_of(ctx->lm.packed, M, c.vocab, d, pf_depth);
            int rc_ = launch_gemm(ctx, kResid, lw.dn, a, F, l + 1 < c.n_layers ? dv.Nqkv : c.vocab);
            if (rc_) return rc_;
        }
    }
    if (want_logits) {
        ctx->n_launch += 1 + (want_reject ? 1 : 0);   // row_stats, accept_sample
        float* logits = ctx->W<float>(ctx->ws.logits);
        RowStat* stats = ctx->W<RowStat>(ctx->ws.stats);
        {
            GemmArgs a = base;
            a.xf = (const uint4*)xf_h; a.N = c.vocab; a.ssq_in = ssqA; a.out = logits;
            int rc_ = launch_gemm(ctx, kPlain, ctx->lm, a, d, 0);
            if (rc_) return rc_;
        }
        // plain launches from here on: they start after the GEMM has fully completed
        row_stats_kernel<<<dim3(M, kStatSplits), 256, 0, st>>>(c.vocab, logits, stats);
        ctx->last_rows = M;
        if (want_reject) {
            CU(launch_pdl_cluster(accept_sample_kernel, dim3(kSampleCluster, n_items), dim3(kSampleThreads), 0, st,
                                  kSampleCluster, (const float*)logits, c.vocab, (const RowStat*)stats,
                                  reinterpret_cast<const RejectItem*>(ctx->wsp + ctx->ws.meta + ml.rej), meta.row_tok,
                                  reinterpret_cast<const float*>(ctx->wsp + ctx->ws.meta + ml.u),
                                  ctx->W<RejectOut>(ctx->ws.results), ctx->W<ReqState>(ctx->ws.req_state)));
        }
    }
    CU(cudaGetLastError());
    return PIPESD_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------- C ABI
extern "C" {

const char* pipesd_strerror(int32_t s) {
    switch (s) {
        case PIPESD_OK: return "ok";
        case PIPESD_E_INVALID: return "invalid argument";
        case PIPESD_E_FULL: return "no free request slot";
        case PIPESD_E_OOM_PAGES: return "KV page pool exhausted";
        case PIPESD_E_STATE: return "call order violated";
        case PIPESD_E_RANGE: return "length out of range";
        case PIPESD_E_CUDA: return "CUDA failure";
        case PIPESD_E_NOMEM: return "caller buffer too small";
        case PIPESD_E_TOO_LARGE: return "problem needs more scratch than the library's built-in array holds";
        default: return "unknown status";
    }
}

const char* pipesd_last_error(const pipesd_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int32_t pipesd_query_sizes(const pipesd_model_cfg* cfg, pipesd_sizes* out) {
    int rc = check_cfg(cfg);
    if (rc != PIPESD_OK || !out) return PIPESD_E_INVALID;
    Derived d = derive(*cfg);
    out->weights_bytes = weights_bytes(*cfg, d);
    out->kv_bytes = kv_bytes(*cfg);
    out->workspace_bytes = ws_layout(*cfg, d).total;
    return PIPESD_OK;
}

int32_t pipesd_ctx_create(const pipesd_model_cfg* cfg, const pipesd_weights* w, const pipesd_mem* mem,
                          void* cuda_stream, pipesd_ctx** out) {
    int rc = check_cfg(cfg);
    if (rc != PIPESD_OK) return rc;
    if (!w || !mem || !out || !w->tok_emb || !w->lm_head || !w->final_norm || !w->layers) return PIPESD_E_INVALID;
    if (!mem->weights || !mem->kv || !mem->workspace) return PIPESD_E_INVALID;
    pipesd_ctx* ctx = new (std::nothrow) pipesd_ctx();
    if (!ctx) return PIPESD_E_INVALID;
    ctx->cfg = *cfg;
    ctx->dv = derive(*cfg);
    ctx->ws = ws_layout(*cfg, ctx->dv);
    ctx->ml = meta_layout(cfg->max_rows, ctx->dv.max_items);
    ctx->st = (cudaStream_t)cuda_stream;
    const pipesd_model_cfg& c = ctx->cfg;
    const Derived& dv = ctx->dv;
    auto bail = [&](int code) { pipesd_ctx_destroy(ctx); return code; };
    if (mem->weights_bytes < weights_bytes(c, dv) || mem->kv_bytes < kv_bytes(c) ||
        mem->workspace_bytes < ctx->ws.total)
        return bail(PIPESD_E_NOMEM);
    if (((uintptr_t)mem->weights | (uintptr_t)mem->kv | (uintptr_t)mem->workspace) & 255) return bail(PIPESD_E_INVALID);
    cudaError_t e = cudaSetDevice(c.device);
    if (e != cudaSuccess) return bail(PIPESD_E_CUDA);
    if (ensure_device_ready() != PIPESD_OK) return bail(PIPESD_E_CUDA);

    {   // CTAs of the attention kernel the device keeps resident at once, per footprint: the key-split plan of a request
        // aims at one wave.  Counted here from the limits that bind (shared memory, registers, threads, tensor-memory
        // columns): the runtime's occupancy query answers one CTA per SM for any kernel that allocates tensor memory.
        int n_sm = 0, smem_sm = 0, smem_rsv = 0, regs_sm = 0, thr_sm = 0;
        if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, c.device) != cudaSuccess || n_sm < 1 ||
            cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, c.device) != cudaSuccess ||
            cudaDeviceGetAttribute(&smem_rsv, cudaDevAttrReservedSharedMemoryPerBlock, c.device) != cudaSuccess ||
            cudaDeviceGetAttribute(&regs_sm, cudaDevAttrMaxRegistersPerMultiprocessor, c.device) != cudaSuccess ||
            cudaDeviceGetAttribute(&thr_sm, cudaDevAttrMaxThreadsPerMultiProcessor, c.device) != cudaSuccess)
            return bail(PIPESD_E_CUDA);
        ctx->n_sm = n_sm;
        cudaFuncAttributes fa;
        if (cudaFuncGetAttributes(&fa, c.head_dim == 128 ? (const void*)attn_kernel<128> : (const void*)attn_kernel<64>) != cudaSuccess)
            return bail(PIPESD_E_CUDA);
        // registers: allocated per warp (in units of 512), and a CTA's warps are dealt to the SM's four register
        // partitions in turn, so the fullest partition binds
        const int regs_warp = (fa.numRegs * 32 + 511) / 512 * 512;
        const int warps_part = (kAttnThreads / 32 + 3) / 4;
        for (int qt = 1; qt <= kAttnMaxRows / 16; ++qt)
            for (int short_tail = 0; short_tail < 2; ++short_tail) {
                const size_t smem_cta = attn_smem_bytes(c.head_dim, 16 * qt, short_tail != 0) + fa.sharedSizeBytes + smem_rsv;
                int per_sm = (int)(smem_sm / smem_cta);
                per_sm = std::min(per_sm, (regs_sm / 4) / std::max(1, regs_warp * warps_part));
                per_sm = std::min(per_sm, thr_sm / kAttnThreads);
                per_sm = std::min(per_sm, 512 / attn_tmem_cols(16 * qt));
                ctx->attn_slots[qt][short_tail] = std::max(1, per_sm) * n_sm;
            }
    }
    ctx->kv_pool = (uint16_t*)mem->kv;
    ctx->wsp = (char*)mem->workspace;
    for (int i = 0; i < pipesd_ctx::kStages; ++i) {
        if (cudaHostAlloc((void**)&ctx->h_meta[i], ctx->ml.total, cudaHostAllocDefault) != cudaSuccess)
            return bail(PIPESD_E_CUDA);
        if (cudaEventCreateWithFlags(&ctx->ev_meta[i], cudaEventDisableTiming) != cudaSuccess)
            return bail(PIPESD_E_CUDA);
    }
    for (int i = 0; i < pipesd_ctx::kStages; ++i)
        if (cudaHostAlloc((void**)&ctx->h_results[i], sizeof(RejectOut) * dv.max_items + 16, cudaHostAllocDefault) != cudaSuccess)
            return bail(PIPESD_E_CUDA);

    cudaStream_t st = ctx->st;
    // the device error word and the attention tickets start at zero (the tickets reset themselves after use)
    if (cudaMemsetAsync(ctx->err_word(), 0, 4, st) != cudaSuccess) return bail(PIPESD_E_CUDA);
    if (cudaMemsetAsync(ctx->wsp + ctx->ws.tickets, 0, 4 * (size_t)c.max_rows * c.n_q_heads, st) != cudaSuccess)
        return bail(PIPESD_E_CUDA);

    // ---- repack the weights into the library's own layout
    char* wp = (char*)mem->weights;
    size_t off = 0;
    auto take = [&](size_t bytes) { char* p = wp + off; off += align_up(bytes); return p; };
    auto pack = [&](GemmW& g, int N, int K, int mode, std::initializer_list<std::pair<const void*, int>> srcs) {
        g.N = N;
        g.K = K;
        PackSrc ps = {};
        ps.mode = mode;
        ps.hd = c.head_dim;
        int i = 0;
        for (auto& s : srcs) { ps.w[i] = (const uint16_t*)s.first; ps.rows[i] = s.second; ++i; }
        size_t total = (size_t)((N + 127) / 128 * 8) * (K / 16) * 32;
        int blocks = (int)std::min<size_t>((total + 255) / 256, 148 * 16);
        g.packed = (uint4*)take(gemm_packed_bytes(N, K));
        gemm_pack_kernel<<<blocks, 256, 0, st>>>(ps, g.packed, N, K);
        if (c.max_rows > 32) {
            g.packed_u = (uint4*)take(gemm_packed_bytes(N, K));
            gemm_pack_umma_kernel<<<blocks, 256, 0, st>>>(ps, g.packed_u, N, K);
        }
    };
    ctx->emb = (uint16_t*)take((size_t)c.vocab * c.d_model * 2);
    if (cudaMemcpyAsync(ctx->emb, w->tok_emb, (size_t)c.vocab * c.d_model * 2, cudaMemcpyDeviceToDevice, st) !=
        cudaSuccess)
        return bail(PIPESD_E_CUDA);
    ctx->layers.resize(c.n_layers);
    for (int l = 0; l < c.n_layers; ++l) {
        const pipesd_layer_weights& s = w->layers[l];
        if (!s.wq || !s.wk || !s.wv || !s.wo || !s.wg || !s.wu || !s.wd || !s.attn_norm || !s.ffn_norm)
            return bail(PIPESD_E_INVALID);
        LayerW& lw = ctx->layers[l];
        pack(lw.qkv, dv.Nqkv, c.d_model, kQkvRope, {{s.wq, dv.qd}, {s.wk, dv.kvd}, {s.wv, dv.kvd}});
        pack(lw.o, c.d_model, dv.qd, kPlain, {{s.wo, c.d_model}});
        pack(lw.gu, 2 * c.d_ffn, c.d_model, kSwiglu, {{s.wg, c.d_ffn}, {s.wu, c.d_ffn}});
        pack(lw.dn, c.d_model, c.d_ffn, kPlain, {{s.wd, c.d_model}});
        lw.n1 = (float*)take(4 * (size_t)c.d_model);
        lw.n2 = (float*)take(4 * (size_t)c.d_model);
        cudaMemcpyAsync(lw.n1, s.attn_norm, 4 * (size_t)c.d_model, cudaMemcpyDeviceToDevice, st);
        cudaMemcpyAsync(lw.n2, s.ffn_norm, 4 * (size_t)c.d_model, cudaMemcpyDeviceToDevice, st);
    }
    pack(ctx->lm, c.vocab, c.d_model, kPlain, {{w->lm_head, c.vocab}});
    ctx->final_norm = (float*)take(4 * (size_t)c.d_model);
    cudaMemcpyAsync(ctx->final_norm, w->final_norm, 4 * (size_t)c.d_model, cudaMemcpyDeviceToDevice, st);
    if (cudaGetLastError() != cudaSuccess) return bail(PIPESD_E_CUDA);

    ctx->reqs.resize(c.max_requests);
    ctx->free_pages.resize(c.n_pages);
    for (int i = 0; i < c.n_pages; ++i) ctx->free_pages[i] = c.n_pages - 1 - i;
    *out = ctx;
    return PIPESD_OK;
}

int32_t pipesd_ctx_destroy(pipesd_ctx* ctx) {
    if (!ctx) return PIPESD_E_INVALID;
    if (ctx->wsp) cudaStreamSynchronize(ctx->st);
    for (int i = 0; i < pipesd_ctx::kStages; ++i) {
        if (ctx->h_meta[i]) cudaFreeHost(ctx->h_meta[i]);
        if (ctx->ev_meta[i]) cudaEventDestroy(ctx->ev_meta[i]);
    }
    for (int i = 0; i < pipesd_ctx::kStages; ++i)
        if (ctx->h_results[i]) cudaFreeHost(ctx->h_results[i]);
    for (cudaEvent_t e : ctx->prof_ev) cudaEventDestroy(e);
    delete ctx;
    return PIPESD_OK;
}

int32_t pipesd_ctx_sync(pipesd_ctx* ctx) {
    if (!ctx) return PIPESD_E_INVALID;
    CU(cudaStreamSynchronize(ctx->st));
    if (ctx->inflight.empty()) return PIPESD_OK;
    // The device error word travels with every call's results; the kernels only ever set it, so the newest copy
    // tells whether any bounded device-side wait of the calls in flight gave up.
    const int dev_err = *reinterpret_cast<const int*>(ctx->h_results[ctx->inflight.back().buf] + ctx->dv.max_items);
    if (dev_err) {   // the results of every call in flight are void; nothing is committed
        for (const pipesd_ctx::Inflight& f : ctx->inflight) {
            for (size_t i = 0; i < f.items.size(); ++i) {
                if (f.dst) f.dst[i].status = PIPESD_E_CUDA;
                if (f.items[i].commit != kCommitNone) ctx->reqs[f.items[i].slot].spec = 0;
            }
        }
        ctx->inflight.clear();
        cudaMemsetAsync(ctx->err_word(), 0, 4, ctx->st);
        cudaMemsetAsync(ctx->wsp + ctx->ws.tickets, 0, 4 * (size_t)ctx->cfg.max_rows * ctx->cfg.n_q_heads, ctx->st);
        char msg[96];
        snprintf(msg, sizeof msg, "a device-side wait timed out (kernel error word %d)", dev_err);
        return fail(ctx, PIPESD_E_CUDA, msg);
    }
    for (const pipesd_ctx::Inflight& f : ctx->inflight) {
        const RejectOut* res = ctx->h_results[f.buf];
        for (size_t i = 0; i < f.items.size(); ++i) {
            if (f.dst) {
                f.dst[i].n_accepted = res[i].n_accepted;
                f.dst[i].next_token = res[i].next_token;
                f.dst[i].status = res[i].status;
                f.dst[i].reserved = 0;
            }
            const pipesd_ctx::InflightItem& it = f.items[i];
            if (it.commit == kCommitNone) continue;
            // what the kernel committed on the device, applied to the host's bookkeeping (calls in order)
            Request& r = ctx->reqs[it.slot];
            r.spec -= it.k + 1;
            if (res[i].status == 0) {
                r.len += 1 + res[i].n_accepted;
                r.pending = res[i].next_token;
            }
            if (r.spec == 0) shrink_pages(ctx, r, r.len);
        }
    }
    ctx->inflight.clear();
    return PIPESD_OK;
}

int32_t pipesd_req_open(pipesd_ctx* ctx, int32_t* req) {
    if (!ctx || !req) return PIPESD_E_INVALID;
    for (int i = 0; i < (int)ctx->reqs.size(); ++i)
        if (!ctx->reqs[i].open) {
            ctx->reqs[i] = Request();
            ctx->reqs[i].open = true;
            *req = i;
            return PIPESD_OK;
        }
    return fail(ctx, PIPESD_E_FULL, "pipesd_req_open");
}

static inline bool bad_req(const pipesd_ctx* ctx, int32_t req) {
    return req < 0 || req >= (int)ctx->reqs.size() || !ctx->reqs[req].open;
}

int32_t pipesd_req_close(pipesd_ctx* ctx, int32_t req) {
    if (!ctx || bad_req(ctx, req)) return fail(ctx, PIPESD_E_INVALID, "pipesd_req_close: bad request");
    Request& r = ctx->reqs[req];
    shrink_pages(ctx, r, 0);
    r = Request();
    return PIPESD_OK;
}

int32_t pipesd_req_len(pipesd_ctx* ctx, int32_t req, int32_t* len) {
    if (!ctx || !len || bad_req(ctx, req)) return fail(ctx, PIPESD_E_INVALID, "pipesd_req_len: bad request");
    *len = ctx->reqs[req].len;
    return PIPESD_OK;
}

int32_t pipesd_prefill(pipesd_ctx* ctx, int32_t req, const int32_t* tokens, int32_t n, float* last_logits) {
    if (!ctx || !tokens || n < 1 || bad_req(ctx, req)) return fail(ctx, PIPESD_E_INVALID, "pipesd_prefill");
    Request& r = ctx->reqs[req];
    if (r.tentative || r.spec) return fail(ctx, PIPESD_E_STATE, "prefill on a request with an uncommitted verify");
    if ((int)ctx->inflight.size() >= pipesd_ctx::kStages) {
        int rc0 = pipesd_ctx_sync(ctx);
        if (rc0 != PIPESD_OK) return rc0;
    }
    if (r.len + n > ctx->cfg.max_seq) return fail(ctx, PIPESD_E_RANGE, "prefill beyond max_seq");
    for (int i = 0; i < n; ++i)
        if (tokens[i] < 0 || tokens[i] >= ctx->cfg.vocab) return fail(ctx, PIPESD_E_INVALID, "token id out of range");
    if (pages_needed(ctx, r, r.len + n) > (int)ctx->free_pages.size())
        return fail(ctx, PIPESD_E_OOM_PAGES, "pipesd_prefill");
    int rc = grow_pages(ctx, req, r.len + n);
    if (rc != PIPESD_OK) return rc;
    const int chunk = std::min(ctx->cfg.max_rows, kMaxItemRows);
    for (int done = 0; done < n; done += chunk) {
        int rows = std::min(chunk, n - done);
        bool last = done + rows == n;
        std::vector<ItemDesc> items(1);
        items[0] = ItemDesc{req, rows, 2, 0, tokens + done, nullptr, nullptr, r.len, kCommitNone, 0};
        rc = run_pass(ctx, items, last && last_logits, false);
        if (rc != PIPESD_OK) return rc;
        r.len += rows;
        r.pending = -1;
        if (last) {   // the device error word travels back with the (unused) result slots; pipesd_ctx_sync reads it
            rc = push_inflight(ctx, nullptr, {});
            if (rc != PIPESD_OK) return rc;
        }
        if (last && last_logits) {
            CU(cudaMemcpyAsync(last_logits, ctx->W<float>(ctx->ws.logits) + (size_t)(rows - 1) * ctx->cfg.vocab,
                               4 * (size_t)ctx->cfg.vocab, cudaMemcpyDeviceToHost, ctx->st));
            rc = pipesd_ctx_sync(ctx);
            if (rc != PIPESD_OK) return rc;
        }
    }
    return PIPESD_OK;
}

int32_t pipesd_verify(pipesd_ctx* ctx, int32_t n_req, const pipesd_verify_item* items_in,
                      pipesd_verify_result* results, uint32_t flags) {
    if (!ctx || !items_in || !results || n_req < 1 || n_req > ctx->dv.max_items)
        return fail(ctx, PIPESD_E_INVALID, "pipesd_verify: arguments");
    if (flags & ~(uint32_t)(PIPESD_Q_HOST | PIPESD_AUTOCOMMIT | PIPESD_CHAIN))
        return fail(ctx, PIPESD_E_INVALID, "pipesd_verify: unknown flag");
    const pipesd_model_cfg& c = ctx->cfg;
    const bool chain = (flags & PIPESD_CHAIN) != 0;
    const int commit = chain ? kCommitChain : ((flags & PIPESD_AUTOCOMMIT) ? kCommitAuto : kCommitNone);
    // A chained call rides behind the calls in flight; any other call first takes delivery of their results (the host
    // needs the committed lengths), and so does a chained one once every staging buffer is taken.
    if (!ctx->inflight.empty() && (!chain || (int)ctx->inflight.size() >= pipesd_ctx::kStages)) {
        int rc = pipesd_ctx_sync(ctx);
        if (rc != PIPESD_OK) return rc;
    }
    int M = 0, pages = 0;
    std::vector<char> seen(c.max_requests, 0);
    for (int i = 0; i < n_req; ++i) {
        const pipesd_verify_item& it = items_in[i];
        if (bad_req(ctx, it.req) || seen[it.req]) return fail(ctx, PIPESD_E_INVALID, "verify: bad or repeated request");
        seen[it.req] = 1;
        if (it.k < 1 || it.k > c.max_draft || !it.tokens) return fail(ctx, PIPESD_E_INVALID, "verify: item");
        if (it.mode == PIPESD_MODE_STOCHASTIC && !it.u) return fail(ctx, PIPESD_E_INVALID, "verify: uniforms missing");
        if (it.mode != PIPESD_MODE_STOCHASTIC && it.mode != PIPESD_MODE_GREEDY)
            return fail(ctx, PIPESD_E_INVALID, "verify: mode");
        if (it.mode == PIPESD_MODE_STOCHASTIC && !it.q) return fail(ctx, PIPESD_E_INVALID, "verify: q missing");
        const Request& r = ctx->reqs[it.req];
        for (int j = 0; j <= it.k; ++j) {
            const bool use_pending = j == 0 && it.tokens[0] == PIPESD_TOKEN_PENDING && !chain;
            if (use_pending && r.pending < 0) return fail(ctx, PIPESD_E_STATE, "verify: no pending token recorded for the request");
            if (!use_pending && (it.tokens[j] < 0 || it.tokens[j] >= c.vocab)) return fail(ctx, PIPESD_E_INVALID, "verify: token id");
            if (it.u && !(it.u[j] >= 0.f && it.u[j] < 1.f)) return fail(ctx, PIPESD_E_INVALID, "verify: uniform outside [0,1)");
        }
        if (r.tentative) return fail(ctx, PIPESD_E_STATE, "verify on a request with an uncommitted tail");
        if (chain && !r.spec) return fail(ctx, PIPESD_E_STATE, "chained verify without a commit-on-device verify in flight");
        if (!chain && r.spec) return fail(ctx, PIPESD_E_STATE, "verify on a request with an uncommitted tail");
        if (r.len + r.spec + it.k + 1 > c.max_seq) return fail(ctx, PIPESD_E_RANGE, "verify beyond max_seq");
        M += it.k + 1;
        pages += pages_needed(ctx, r, r.len + r.spec + it.k + 1);
    }
    if (M > c.max_rows) return fail(ctx, PIPESD_E_RANGE, "verify: more rows than max_rows");
    if (pages > (int)ctx->free_pages.size()) return fail(ctx, PIPESD_E_OOM_PAGES, "pipesd_verify");

    std::vector<ItemDesc> items(n_req);
    std::vector<pipesd_ctx::InflightItem> fl(n_req);
    float* qstage = ctx->W<float>(ctx->ws.qstage);
    size_t qrow = 0;
    for (int i = 0; i < n_req; ++i) {
        const pipesd_verify_item& it = items_in[i];
        const Request& r = ctx->reqs[it.req];
        const int base = r.len + r.spec;      // a chained pass is planned as if its predecessors had accepted every draft
        int rc = grow_pages(ctx, it.req, base + it.k + 1);
        if (rc != PIPESD_OK) return rc;
        const float* q = it.q;
        if (it.mode == PIPESD_MODE_STOCHASTIC && (flags & PIPESD_Q_HOST)) {
            float* dst = qstage + qrow * c.vocab;
            CU(cudaMemcpyAsync(dst, it.q, 4 * (size_t)it.k * c.vocab, cudaMemcpyHostToDevice, ctx->st));
            q = dst;
            qrow += it.k;
        }
        items[i] = ItemDesc{it.req, it.k + 1, it.mode, it.k, it.tokens, q, it.u, base, commit, r.pending};
        fl[i] = pipesd_ctx::InflightItem{it.req, it.k, commit};
    }
    int rc = run_pass(ctx, items, true, true);
    if (rc != PIPESD_OK) return rc;
    rc = push_inflight(ctx, results, std::move(fl));
    if (rc != PIPESD_OK) return rc;
    for (int i = 0; i < n_req; ++i) {
        Request& r = ctx->reqs[items_in[i].req];
        if (commit == kCommitNone) r.tentative = items_in[i].k + 1;
        else r.spec += items_in[i].k + 1;
    }
    return PIPESD_OK;
}

int32_t pipesd_kv_rollback(pipesd_ctx* ctx, int32_t n_req, const int32_t* reqs, const int32_t* n_accepted,
                           const int32_t* next_token) {
    if (!ctx || !reqs || !n_accepted || n_req < 1) return fail(ctx, PIPESD_E_INVALID, "pipesd_kv_rollback");
    std::vector<char> seen(ctx->cfg.max_requests, 0);
    for (int i = 0; i < n_req; ++i) {
        if (bad_req(ctx, reqs[i])) return fail(ctx, PIPESD_E_INVALID, "rollback: bad request");
        if (seen[reqs[i]]) return fail(ctx, PIPESD_E_INVALID, "rollback: repeated request");
        seen[reqs[i]] = 1;
        const Request& r = ctx->reqs[reqs[i]];
        if (!r.tentative) return fail(ctx, PIPESD_E_STATE, "rollback without a preceding verify");
        if (n_accepted[i] < 0 || n_accepted[i] > r.tentative - 1)
            return fail(ctx, PIPESD_E_RANGE, "rollback: n_accepted outside 0..k");
        if (next_token && (next_token[i] < 0 || next_token[i] >= ctx->cfg.vocab))
            return fail(ctx, PIPESD_E_INVALID, "rollback: next_token is not a token id");
    }
    for (int i = 0; i < n_req; ++i) {
        Request& r = ctx->reqs[reqs[i]];
        r.len += 1 + n_accepted[i];
        r.tentative = 0;
        r.pending = next_token ? next_token[i] : -1;
        shrink_pages(ctx, r, r.len);
    }
    return PIPESD_OK;
}

int32_t pipesd_debug_get_logits(pipesd_ctx* ctx, float* dst, int32_t rows) {
    if (!ctx || !dst || rows < 1 || rows > ctx->last_rows) return fail(ctx, PIPESD_E_INVALID, "pipesd_debug_get_logits");
    CU(cudaMemcpyAsync(dst, ctx->W<float>(ctx->ws.logits), 4 * (size_t)rows * ctx->cfg.vocab, cudaMemcpyDeviceToHost,
                       ctx->st));
    CU(cudaStreamSynchronize(ctx->st));
    return PIPESD_OK;
}

static int32_t kv_rw(pipesd_ctx* ctx, int32_t req, int32_t layer, int32_t pos0, int32_t n_pos, uint16_t* k,
                     uint16_t* v, bool write) {
    if (!ctx || !k || !v || bad_req(ctx, req) || layer < 0 || layer >= ctx->cfg.n_layers || pos0 < 0 || n_pos < 1)
        return fail(ctx, PIPESD_E_INVALID, "kv read/write");
    const pipesd_model_cfg& c = ctx->cfg;
    Request& r = ctx->reqs[req];
    if (r.tentative || r.spec) return fail(ctx, PIPESD_E_STATE, "kv read/write with an uncommitted verify");
    const int end = pos0 + n_pos;
    if (write) {
        if (end > c.max_seq) return fail(ctx, PIPESD_E_RANGE, "kv write beyond max_seq");
        if (pages_needed(ctx, r, end) > (int)ctx->free_pages.size()) return fail(ctx, PIPESD_E_OOM_PAGES, "kv write");
        int rc = grow_pages(ctx, req, end);
        if (rc != PIPESD_OK) return rc;
        r.len = std::max(r.len, end);
    } else if (end > r.len) {
        return fail(ctx, PIPESD_E_RANGE, "kv read beyond the committed length");
    }
    const int w = ctx->dv.kvd;
    // staging: the two split-K partial arrays (idle between passes)
    uint16_t* sk = ctx->W<uint16_t>(ctx->ws.partA);
    uint16_t* sv = ctx->W<uint16_t>(ctx->ws.partB);
    const size_t cap = ctx->dv.part_floats * 2 / w;  // positions per round
    if (cap < 1) return fail(ctx, PIPESD_E_NOMEM, "kv staging");
    const int32_t* bt = ctx->W<int32_t>(ctx->ws.block_tab) + (size_t)req * ctx->dv.max_pages;
    const int step = (int)std::min<size_t>(cap, (size_t)1 << 20);
    for (int done = 0; done < n_pos; done += step) {
        int n = std::min(step, n_pos - done);
        size_t bytes = (size_t)n * w * 2;
        if (write) {
            CU(cudaMemcpyAsync(sk, k + (size_t)done * w, bytes, cudaMemcpyHostToDevice, ctx->st));
            CU(cudaMemcpyAsync(sv, v + (size_t)done * w, bytes, cudaMemcpyHostToDevice, ctx->st));
        }
        int blocks = (int)std::min<size_t>(((size_t)n * w + 255) / 256, 148 * 8);
        kv_copy_kernel<<<blocks, 256, 0, ctx->st>>>(ctx->kv_pool, sk, sv, bt, pos0 + done, n, layer, c.n_pages,
                                                    c.page_size, c.n_kv_heads, c.head_dim, write ? 1 : 0);
        if (!write) {
            CU(cudaMemcpyAsync(k + (size_t)done * w, sk, bytes, cudaMemcpyDeviceToHost, ctx->st));
            CU(cudaMemcpyAsync(v + (size_t)done * w, sv, bytes, cudaMemcpyDeviceToHost, ctx->st));
        }
        CU(cudaStreamSynchronize(ctx->st));
    }
    return PIPESD_OK;
}

int32_t pipesd_debug_read_kv(pipesd_ctx* ctx, int32_t req, int32_t layer, int32_t pos0, int32_t n_pos, uint16_t* k,
                             uint16_t* v) {
    return kv_rw(ctx, req, layer, pos0, n_pos, k, v, false);
}

int32_t pipesd_debug_write_kv(pipesd_ctx* ctx, int32_t req, int32_t layer, int32_t pos0, int32_t n_pos,
                              const uint16_t* k, const uint16_t* v) {
    return kv_rw(ctx, req, layer, pos0, n_pos, const_cast<uint16_t*>(k), const_cast<uint16_t*>(v), true);
}

int32_t pipesd_reject_from_logits(pipesd_ctx* ctx, int32_t k, int32_t mode, const float* logits, const float* q,
                                  const int32_t* drafts, const float* u, pipesd_verify_result* result) {
    if (!ctx || !logits || !drafts || !u || !result || k < 1 || k > ctx->cfg.max_draft)
        return fail(ctx, PIPESD_E_INVALID, "pipesd_reject_from_logits");
    if (mode != PIPESD_MODE_GREEDY && (mode != PIPESD_MODE_STOCHASTIC || !q))
        return fail(ctx, PIPESD_E_INVALID, "pipesd_reject_from_logits: mode / q");
    if (!ctx->inflight.empty()) {
        int rc = pipesd_ctx_sync(ctx);
        if (rc != PIPESD_OK) return rc;
    }
    const int V = ctx->cfg.vocab;
    for (int i = 0; i < k; ++i)
        if (drafts[i] < 0 || drafts[i] >= V) return fail(ctx, PIPESD_E_INVALID, "draft id out of range");
    const int sidx = ctx->stage;
    ctx->stage = (ctx->stage + 1) % pipesd_ctx::kStages;
    CU(cudaEventSynchronize(ctx->ev_meta[sidx]));
    char* hm = ctx->h_meta[sidx];
    const MetaLayout& ml = ctx->ml;
    int32_t* tok = reinterpret_cast<int32_t*>(hm + ml.row_tok);
    tok[0] = 0;
    for (int i = 0; i < k; ++i) tok[i + 1] = drafts[i];
    float* hu = reinterpret_cast<float*>(hm + ml.u);
    for (int i = 0; i <= k; ++i) hu[i] = u[i];
    float* dl = ctx->W<float>(ctx->ws.logits);
    float* dq = ctx->W<float>(ctx->ws.qstage);
    RejectItem* hr = reinterpret_cast<RejectItem*>(hm + ml.rej);
    hr[0] = RejectItem{0, k, mode, 0, dq, 0, 0, kCommitNone, 0};
    cudaStream_t st = ctx->st;
    CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.meta, hm, ml.total, cudaMemcpyHostToDevice, st));
    CU(cudaEventRecord(ctx->ev_meta[sidx], st));
    CU(cudaMemcpyAsync(dl, logits, 4 * (size_t)(k + 1) * V, cudaMemcpyHostToDevice, st));
    if (mode == PIPESD_MODE_STOCHASTIC) CU(cudaMemcpyAsync(dq, q, 4 * (size_t)k * V, cudaMemcpyHostToDevice, st));
    RowStat* stats = ctx->W<RowStat>(ctx->ws.stats);
    row_stats_kernel<<<dim3(k + 1, kStatSplits), 256, 0, st>>>(V, dl, stats);
    CU(cudaGetLastError());
    CU(launch_pdl_cluster(accept_sample_kernel, dim3(kSampleCluster, 1), dim3(kSampleThreads), 0, st, kSampleCluster,
                          (const float*)dl, V, (const RowStat*)stats,
                          reinterpret_cast<const RejectItem*>(ctx->wsp + ctx->ws.meta + ml.rej),
                          reinterpret_cast<const int32_t*>(ctx->wsp + ctx->ws.meta + ml.row_tok),
                          reinterpret_cast<const float*>(ctx->wsp + ctx->ws.meta + ml.u),
                          ctx->W<RejectOut>(ctx->ws.results), ctx->W<ReqState>(ctx->ws.req_state)));
    RejectOut* hres = ctx->h_results[0];   // nothing is in flight here (synchronised above)
    CU(cudaMemcpyAsync(hres, ctx->W<RejectOut>(ctx->ws.results), sizeof(RejectOut), cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    result->n_accepted = hres[0].n_accepted;
    result->next_token = hres[0].next_token;
    result->status = hres[0].status;
    result->reserved = 0;
    ctx->last_rows = k + 1;
    return PIPESD_OK;
}

int32_t pipesd_debug_set_len(pipesd_ctx* ctx, int32_t req, int32_t new_len) {
    if (!ctx || bad_req(ctx, req)) return fail(ctx, PIPESD_E_INVALID, "pipesd_debug_set_len");
    Request& r = ctx->reqs[req];
    if (r.tentative || r.spec) return fail(ctx, PIPESD_E_STATE, "set_len with an uncommitted verify");
    if (new_len < 0 || new_len > r.len) return fail(ctx, PIPESD_E_RANGE, "set_len can only truncate");
    r.len = new_len;
    r.pending = -1;
    shrink_pages(ctx, r, r.len);
    return PIPESD_OK;
}

int32_t pipesd_debug_req_state(pipesd_ctx* ctx, int32_t req, int32_t* out3) {
    if (!ctx || !out3 || bad_req(ctx, req)) return fail(ctx, PIPESD_E_INVALID, "pipesd_debug_req_state");
    ReqState s;
    CU(cudaMemcpyAsync(&s, ctx->W<ReqState>(ctx->ws.req_state) + req, sizeof s, cudaMemcpyDeviceToHost, ctx->st));
    CU(cudaStreamSynchronize(ctx->st));
    out3[0] = s.len; out3[1] = s.pending; out3[2] = s.all_accepted;
    return PIPESD_OK;
}

int32_t pipesd_debug_wait_timeout(pipesd_ctx* ctx, int32_t limit_us) {
    if (!ctx || limit_us < 1 || limit_us > 100000) return fail(ctx, PIPESD_E_INVALID, "pipesd_debug_wait_timeout");
    if ((int)ctx->inflight.size() >= pipesd_ctx::kStages) {
        int rc = pipesd_ctx_sync(ctx);
        if (rc != PIPESD_OK) return rc;
    }
    CU(cudaMemsetAsync(ctx->wsp + ctx->ws.never_flag, 0, 16, ctx->st));
    wait_never_kernel<<<1, 32, 0, ctx->st>>>(ctx->W<int>(ctx->ws.never_flag), ctx->err_word(), (unsigned long long)limit_us * 1000ull);
    CU(cudaGetLastError());
    return push_inflight(ctx, nullptr, {});
}

int32_t pipesd_profile_enable(pipesd_ctx* ctx, int32_t time_gemms) {
    if (!ctx) return PIPESD_E_INVALID;
    CU(cudaStreamSynchronize(ctx->st));
    ctx->time_gemms = time_gemms != 0;
    ctx->n_launch = ctx->n_gemm = 0;
    ctx->gemm_bytes = 0.0;
    ctx->prof_used = 0;
    return PIPESD_OK;
}

int32_t pipesd_profile_read(pipesd_ctx* ctx, pipesd_profile_info* out) {
    if (!ctx || !out) return PIPESD_E_INVALID;
    CU(cudaStreamSynchronize(ctx->st));
    double ms = 0.0;
    for (size_t i = 0; i + 1 < ctx->prof_used; i += 2) {
        float t = 0.f;
        CU(cudaEventElapsedTime(&t, ctx->prof_ev[i], ctx->prof_ev[i + 1]));
        ms += t;
    }
    out->kernel_launches = ctx->n_launch;
    out->gemm_launches = ctx->n_gemm;
    out->gemm_ms = ms;
    out->gemm_bytes = ctx->gemm_bytes;
    ctx->n_launch = ctx->n_gemm = 0;
    ctx->gemm_bytes = 0.0;
    ctx->prof_used = 0;
    return PIPESD_OK;
}

uint64_t pipesd_gemm_packed_bytes(int32_t N, int32_t K) {
    if (N < 16 || K < 16) return 0;
    return gemm_packed_bytes(N, K);
}

static size_t gemm_xf_bytes(int M, int K) { return align_up(xf_elems(M, K) * 16); }

uint64_t pipesd_gemm_scratch_bytes(int32_t M, int32_t N, int32_t K) {
    if (M < 1 || N < 16 || K < 16) return 0;
    return gemm_xf_bytes(M, K);
}

int32_t pipesd_gemm_pack(const void* W, void* packed, int32_t N, int32_t K, void* cuda_stream) {
    if (!W || !packed || N < 16 || K < 16 || N % 16 || K % 16) return PIPESD_E_INVALID;
    PackSrc ps = {};
    ps.mode = kPlain;
    ps.w[0] = (const uint16_t*)W;
    ps.rows[0] = N;
    size_t total = (size_t)((N + 127) / 128 * 8) * (K / 16) * 32;
    int blocks = (int)std::min<size_t>((total + 255) / 256, 148 * 16);
    gemm_pack_kernel<<<blocks, 256, 0, (cudaStream_t)cuda_stream>>>(ps, (uint4*)packed, N, K);
    return cudaGetLastError() == cudaSuccess ? PIPESD_OK : PIPESD_E_CUDA;
}

// x -> split-bf16 fragments (the scratch), then the GEMM; the K slices are summed inside the kernel.
static int32_t gemm_run_with_scratch(const void* packed, const float* x, float* y, void* scratch, int M, int N, int K,
                                     cudaStream_t st) {
    const GemmPlan p = gemm_plan(M, N, K);
    uint32_t* xf = (uint32_t*)scratch;
    {
        size_t n = (size_t)M * (K / 2);
        int blocks = (int)std::min<size_t>((n + 255) / 256, 148 * 8);
        xf_format_kernel<<<blocks, 256, 0, st>>>(x, xf, M, K);
    }
    GemmArgs a = {};
    a.W = (const uint4*)packed;
    a.xf = (const uint4*)xf;
    a.M = M;
    a.N = N;
    a.out = y;
    if (gemm_launch(kPlain, p, a, st) != cudaSuccess) return PIPESD_E_CUDA;
    return cudaGetLastError() == cudaSuccess ? PIPESD_OK : PIPESD_E_CUDA;
}

int32_t pipesd_gemm_run(const void* packed, const float* x, float* y, void* scratch, int32_t M, int32_t N,
                        int32_t K, void* cuda_stream) {
    if (!packed || !x || !y || !scratch || M < 1 || N < 16 || K < 16 || N % 16 || K % 16) return PIPESD_E_INVALID;
    if (ensure_device_ready() != PIPESD_OK) return PIPESD_E_CUDA;
    return gemm_run_with_scratch(packed, x, y, scratch, M, N, K, (cudaStream_t)cuda_stream);
}

int32_t pipesd_debug_force_dense(pipesd_ctx* ctx, int32_t on) {
    if (!ctx) return PIPESD_E_INVALID;
    if (on && ctx->cfg.max_rows <= 32)
        return fail(ctx, PIPESD_E_INVALID, "pipesd_debug_force_dense: the context keeps no weights in the dense kernel's order (max_rows <= 32)");
    ctx->force_dense = on != 0;
    return PIPESD_OK;
}

int32_t pipesd_debug_attn_slots(pipesd_ctx* ctx, int32_t rows_per_kv_head, int32_t* out2) {
    if (!ctx || !out2 || rows_per_kv_head < 1) return fail(ctx, PIPESD_E_INVALID, "pipesd_debug_attn_slots");
    const int qt = attn_rows_n(rows_per_kv_head) / 16;
    out2[0] = ctx->attn_slots[qt][0];
    out2[1] = ctx->attn_slots[qt][1];
    return PIPESD_OK;
}

int32_t pipesd_debug_attn_split(int32_t total_keys, int32_t page_size, const int32_t* resident_ctas, int32_t units,
                                int32_t* out3) {
    if (!resident_ctas || !out3 || total_keys < 1 || page_size < 8 || page_size % 8 || units < 1) return PIPESD_E_INVALID;
    const int slots[2] = {resident_ctas[0], resident_ctas[1]};
    const AttnSplit p = attn_split_plan(total_keys, page_size, units, slots);
    out3[0] = p.splits; out3[1] = p.keys_per_split; out3[2] = p.short_tail;
    return PIPESD_OK;
}

}  // extern "C"

extern "C" {

// ---- GEMM without any caller- or library-side allocation ------------------------------------
// The scratch of pipesd_gemm_run_static (activation fragments) lives in this fixed array.  It is part of the
// library image: every GPU that loads the library keeps these bytes reserved until the process
// exits, which is why the limit is modest.
static __device__ __align__(256) unsigned char g_static_gemm_scratch[PIPESD_STATIC_SCRATCH_BYTES];

namespace {
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {nullptr};   // device address of the array, per device ordinal

// In host code the array's name is only a handle for the runtime, not a device address; the address
// a kernel can use comes from cudaGetSymbolAddress, asked once per device with that device current.
int static_scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PIPESD_E_CUDA;
    if (ensure_device_ready() != PIPESD_OK) return PIPESD_E_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_gemm_scratch) != cudaSuccess || !p) return PIPESD_E_CUDA;
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return PIPESD_OK;
}
}  // namespace

int32_t pipesd_gemm_run_static(const void* packed, const float* x, float* y, int32_t M, int32_t N, int32_t K,
                               void* cuda_stream) {
    if (!packed || !x || !y || M < 1 || N < 16 || K < 16 || N % 16 || K % 16) return PIPESD_E_INVALID;
    if (pipesd_gemm_scratch_bytes(M, N, K) > (uint64_t)PIPESD_STATIC_SCRATCH_BYTES) return PIPESD_E_TOO_LARGE;
    void* scratch = nullptr;
    int rc = static_scratch_for_current_device(&scratch);
    if (rc != PIPESD_OK) return rc;
    // Nothing has to be cleared: every activation fragment the GEMM reads is written by this same call
    // first (padding tokens only feed output columns that are never stored), so the previous call's
    // contents never reach the output.
    return gemm_run_with_scratch(packed, x, y, scratch, M, N, K, (cudaStream_t)cuda_stream);
}

}  // extern "C"
