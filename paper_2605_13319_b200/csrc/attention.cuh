// Multi-query decode attention over a paged bf16 KV cache on the tcgen05 tensor cores: each request contributes a
// short chunk of query rows (the pending token plus its k drafts) that attend to the cached prefix and, causally,
// to each other.  The keys are cut into 8 to 10 splits ("split-K") handled by the CTAs of a thread-block cluster;
// every CTA produces an un-normalised partial output with its reference maximum and sum in its own shared memory,
// and after a cluster barrier the partials are merged over distributed shared memory and written straight into the
// output projection's input format -- no partial results in global memory and no separate merge kernel (requests
// of 4096 keys and more use several clusters and one more merge step).  Tiles of keys that were cached before
// this pass do not depend on the preceding QKV projection, so their copies are issued before the dependent-launch
// wait.
//
// One CTA = one KV head of one request x one key split x up to 128 query rows, where the rows are all (query head
// of the group, chunk row) pairs that share the KV head (GQA).  The keys are on the M side of the MMAs, the (few)
// query rows on the narrow N side:
//   S^T[128 keys x N rows] = K_tile[128 x hd] . Q^T[hd x N]          A = K rows from the cache, B = Q
//   O^T[hd x N rows]      += V_tile^T[hd x 128 keys] . P^T[128 x N]   A = V rows from the cache, B = P
//   L  [  * x N rows]      += 1[* x 128 keys] . P^T[128 x N]          the softmax denominators, by the same P
// with S^T, O^T and L in tensor memory (3N columns).  The cache stores, per page and head, the rows in 8-row groups
// of 8-element pieces ([slot/8][hd/8][slot%8][8]), which IS the operand order of both products (K-major for the
// first, MN-major for the second): a page lands in shared memory by one bulk copy and is read by the tensor cores
// as it is.  Q and P are fp32 values split into bf16 hi + lo terms (two MMAs into the same accumulator); K and V
// are the cache's bf16.
// Warps 0-3 (one thread per key of a tile, i.e. per tensor-memory lane): masking, the running maximum (a row's
// reference maximum only moves when the tile's maximum exceeds it by more than 2^8, so that O^T is rarely
// rescaled), exponentials, P written back as the next MMA's B operand.  Warp 4: bulk copies of the K/V pages and
// the MMA issue (one thread).  Every wait is bounded and raises the device error word.
#pragma once
#include "common.cuh"
#include "layers.cuh"
#include "tcgen05.cuh"

namespace pipesd {

constexpr int kAttnWorkers = 128;           // threads of warps 0-3
constexpr int kAttnThreads = kAttnWorkers + 32;
constexpr int kAttnTile = 128;              // keys per tile = M of the MMAs
constexpr int kAttnMaxRows = 128;           // query rows per CTA (N of the MMAs); more rows: more row groups
constexpr int kAttnPagesSmem = 512;         // page ids of a CTA's key range kept in shared memory (longer ranges read the table)
constexpr float kAttnLazyRescale = 8.f;     // log2 units by which a tile's maximum may exceed the reference maximum

// Wait for a barrier phase.  Bounded by a try count (each try suspends for a hardware-chosen time; 2^22 of them take
// seconds), so that a protocol error cannot hang the GPU: the caller raises the error word and carries on.
__device__ __forceinline__ bool attn_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        uint32_t ok;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}

// The same for a whole warp: every lane waits, and the warp agrees on the outcome (the collective tensor-memory
// instructions that follow need a warp-uniform control flow).
__device__ __forceinline__ bool attn_wait_warp(uint32_t bar, uint32_t parity) {
    return __all_sync(0xffffffffu, attn_wait(bar, parity));
}

__device__ __forceinline__ float fast_exp2(float x) {   // 2^x, relative error 2^-22; 2^-inf = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory plan of one CTA with N query rows (a multiple of 16).
template <int HD>
struct AttnSmem {
    static constexpr int kTileBytes = kAttnTile * HD * 2;            // one K or V tile
    static constexpr int kOnes = 4096;                                // 128 x 16 ones (the denominators' A operand)
    static constexpr int kSmall = 4 * kAttnMaxRows * 4               // warp maxima [4][128]
                                  + 4 * kAttnMaxRows * 4             // horizon, reference maximum, rescale factor, Fl
                                  + 128;                             // barriers, tensor-memory base, flags
    __host__ __device__ static constexpr int q_bytes(int N) { return N * HD * 2; }          // hi or lo
    __host__ __device__ static constexpr int p_bytes(int N) { return kAttnTile * N * 2; }   // hi or lo
    __host__ __device__ static constexpr size_t bytes(int N) {
        return (size_t)2 * kTileBytes + 2 * q_bytes(N) + 2 * p_bytes(N) + kOnes + kSmall;
    }
};

// Tensor-memory columns of a CTA with N query rows: S^T, O^T and L, N columns each, as a power of two >= 32.
__host__ __device__ constexpr int attn_tmem_cols(int N) {
    int c = 32;
    while (c < 3 * N) c *= 2;
    return c;
}
// Dynamic shared memory to ask for: the plan above, padded so that the CTAs an SM can hold never want more than the
// SM's 512 tensor-memory columns together (a CTA that waited for columns held by a CTA waiting at a cluster barrier
// could otherwise wait for ever).
static inline size_t attn_smem_bytes(int hd, int N) {
    const size_t need = hd == 128 ? AttnSmem<128>::bytes(N) : AttnSmem<64>::bytes(N);
    const int max_ctas = 512 / attn_tmem_cols(N);
    const size_t floor_ = (size_t)(227 * 1024) / (max_ctas + 1) + 1;
    return need > floor_ ? need : floor_;
}
static inline int attn_rows_n(int rows_per_kv_head) {    // N of a CTA that holds this many query rows
    const int r = rows_per_kv_head > kAttnMaxRows ? kAttnMaxRows : rows_per_kv_head;
    return (r + 15) / 16 * 16;
}

// Per-CTA constants of the tile copies.
struct AttnCtx {
    const uint16_t* kbase;     // K block of page 0 for this layer and KV head
    const int32_t* bt;         // page ids of the request, indexed from bt_first: shared-memory copy of the CTA's range, or the table
    int bt_first;
    size_t page_stride;        // elements between consecutive pages of a layer
    size_t v_off;              // elements from a K block to the V block of the same page and head
    int page_size;
    int k0, k1;
};

// Issue (one warp) the copies of one 128-key tile: the rows of a page that belong to one KV head are contiguous in
// the pool, already in operand order, so every page the tile touches is one bulk copy of K rows (lanes 0-15, one
// page each) and one of V rows (lanes 16-31), counted in bytes on the barrier.  Whole 8-row groups are copied: the
// rows of the last group at or beyond k1 are masked (K) and cleared (V) by the consumers.
template <int HD>
__device__ __forceinline__ void attn_issue_tile(const AttnCtx& c, uint32_t k_addr, uint32_t v_addr, uint32_t bar, int j0) {
    const int lane = threadIdx.x & 31;
    const int j1 = (min(j0 + kAttnTile, c.k1) + 7) & ~7;
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)(j1 - j0) * (HD * 2) * 2);
    __syncwarp();
    const int kv = lane >> 4;
    for (int pg = lane & 15; ; pg += 16) {
        const int pidx = j0 / c.page_size + pg;                            // page of the request
        const int js = max(j0, pidx * c.page_size), je = min(j1, (pidx + 1) * c.page_size);
        if (js >= je) break;
        const uint16_t* src = c.kbase + (size_t)c.bt[pidx - c.bt_first] * c.page_stride + (kv ? c.v_off : 0) +
                              (size_t)(js - pidx * c.page_size) * HD;
        bulk_g2s((kv ? v_addr : k_addr) + (uint32_t)(js - j0) * (HD * 2), src, (uint32_t)(je - js) * (HD * 2), bar);
    }
}

constexpr int kAttnSplits = 8;        // key splits per cluster of a request whose keys several clusters share
constexpr int kAttnMaxCluster = 10;   // largest cluster along x (above 8: the non-portable sizes, opted into by the host)

// Host: how one request's keys are split.  `resident[w - 8]` = clusters of width w (8, 9, 10) the device keeps
// resident at once for this request's shared-memory footprint (0: width unavailable); `need` = clusters the request
// launches per layer (KV heads x row groups).  One cluster of eight per 2048 keys up to four clusters; a single
// cluster widens to the smallest width that leaves each CTA the fewest 128-key tiles, as long as all the request's
// clusters still run in one wave.  Everything here depends on the request alone, never on its batch.
struct AttnSplit { int clusters, width, keys_per_split; };
static inline AttnSplit attn_split_plan(int total_keys, int page_size, const int* resident, int need) {
    AttnSplit p;
    p.clusters = total_keys / 2048 < 1 ? 1 : (total_keys / 2048 > kMaxSplits / kAttnSplits ? kMaxSplits / kAttnSplits : total_keys / 2048);
    p.width = kAttnSplits;
    auto chunk_of = [&](int splits) {
        const int ch = (total_keys + splits - 1) / splits;
        return (ch + page_size - 1) / page_size * page_size;
    };
    auto tiles_of = [&](int splits) { return (chunk_of(splits) + kAttnTile - 1) / kAttnTile; };
    if (p.clusters == 1)
        for (int w = kAttnSplits + 1; w <= kAttnMaxCluster; ++w)
            if (resident[w - kAttnSplits] >= need && tiles_of(w) < tiles_of(p.width)) p.width = w;
    p.keys_per_split = chunk_of(p.width * p.clusters);
    return p;
}

struct AttnArgs {
    const float* q;            // [M][Hq*hd] rotated queries
    PassMeta meta;
    const uint16_t* kv_pool;
    int layer, n_pages, page_size, M, Hq, Hkv;
    int n_max;                 // N the launch's shared memory was sized for
    int row_groups;
    float* o_part;             // partial results of requests whose keys several clusters share
    float* m_part;
    float* l_part;
    int* tickets;
    uint16_t* xf_out;          // the output projection's input (split-bf16 fragments)
    int* err;
};

// grid (cs * max clusters per request, n_kv_heads * row_groups, n_items), cluster (cs,1,1), 8 <= cs <= 10, block 160.
// A request uses the first it_cs <= cs CTAs of its cluster; the others hold an empty split (exact zeros in the
// merge), so a request's result does not depend on the cluster size its batch was launched with.
// A request whose keys are shared by several clusters (long contexts) takes one more step: every cluster
// writes its merged partial to global memory and the last cluster to arrive (atomic ticket, nobody waits)
// merges those.
template <int HD>
__global__ void __launch_bounds__(kAttnThreads) attn_kernel(const AttnArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    using SM = AttnSmem<HD>;
    constexpr int HG = HD / 8;                                      // 8-element pieces of a row
    pdl_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int item = blockIdx.z;
    const int cs = (int)cluster_nctaid_x();
    const int cl = blockIdx.x / cs, rank = blockIdx.x % cs;        // cluster of this (request, head), rank in it
    const int ncl = a.meta.it_nsplit[item];                        // clusters that share this request's keys
    if (cl >= ncl) return;                                         // taken by a whole cluster or by none
    const int S = a.meta.it_cs[item];                              // key splits per cluster of this request (<= cs)
    const int sp = cl * S + rank;                                  // key split of this CTA (rank < S)
    const int Hkv = a.Hkv, Hq = a.Hq;
    const int kvh = blockIdx.y % Hkv, rg = blockIdx.y / Hkv;
    const int G = Hq / Hkv;
    const int rows = a.meta.it_rows[item];
    const int R = G * rows;
    const int rho0 = rg * kAttnMaxRows;
    // the whole cluster shares (item, head, row group): these exits are taken by all CTAs of the cluster or by none
    if (rho0 >= R) return;
    const int n_rows = min(kAttnMaxRows, R - rho0);
    const int N = (n_rows + 15) & ~15;
    if (N > a.n_max) return;
    const int NG = N / 8;
    const int base = a.meta.it_base[item];
    const int total = base + rows, chunk = a.meta.it_chunk[item];
    AttnCtx c;
    c.k0 = rank < S ? min(sp * chunk, total) : total;
    c.k1 = min(c.k0 + chunk, total);
    c.kbase = a.kv_pool + kv_index(a.layer, a.n_pages, 0, 0, Hkv, kvh, a.page_size, 0, HD, 0);
    c.page_stride = (size_t)2 * Hkv * a.page_size * HD;
    c.v_off = (size_t)Hkv * a.page_size * HD;
    c.page_size = a.page_size;
    c.bt = a.meta.block_tab + (size_t)a.meta.it_slot[item] * a.meta.max_pages;
    c.bt_first = 0;
    const int ntiles = c.k1 > c.k0 ? (c.k1 - c.k0 + kAttnTile - 1) / kAttnTile : 0;

    // ---- shared memory
    unsigned char* k_tile = smem;
    unsigned char* v_tile = k_tile + SM::kTileBytes;
    unsigned char* q_hi = v_tile + SM::kTileBytes;
    unsigned char* q_lo = q_hi + SM::q_bytes(N);
    unsigned char* p_hi = q_lo + SM::q_bytes(N);
    unsigned char* p_lo = p_hi + SM::p_bytes(N);
    unsigned char* ones = p_lo + SM::p_bytes(N);
    float* wm = reinterpret_cast<float*>(ones + SM::kOnes);        // [4][128] warp maxima of a tile
    int* hz = reinterpret_cast<int*>(wm + 4 * kAttnMaxRows);       // [128] last visible key of a row (-1: padding row)
    float* m_ref = reinterpret_cast<float*>(hz + kAttnMaxRows);    // [128] reference maximum of a row
    float* alpha = m_ref + kAttnMaxRows;                           // [128] rescale factor of a row for this tile
    float* Fl = alpha + kAttnMaxRows;                              // [128] the CTA's partial denominators
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(Fl + kAttnMaxRows);   // full, s_full, p_full, pv_done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);
    int* s_flag = reinterpret_cast<int*>(tmem_slot + 1);           // a row's reference maximum moved: rescale
    int* s_last = s_flag + 1;
    float* Fo = reinterpret_cast<float*>(q_hi);                    // [N][HD]: takes over the Q operands after the tile loop
    float* Fm = m_ref;
    const uint32_t bar_full = smem_u32(bars), bar_s = bar_full + 8, bar_p = bar_full + 16, bar_pv = bar_full + 24;
    const uint32_t tmem_cols = (uint32_t)attn_tmem_cols(N);

    __shared__ int s_pages[kAttnPagesSmem];
    __shared__ AttnCtx s_ctx;
    // The page ids of this CTA's key range go to shared memory once: a tile's copies then start without a trip to
    // the block table first.
    if (ntiles > 0) {
        const int p_first = c.k0 / a.page_size, n_pg = (c.k1 - 1) / a.page_size - p_first + 1;
        if (n_pg <= kAttnPagesSmem) {                              // uniform over the CTA
            for (int i = tid; i < n_pg; i += kAttnThreads) s_pages[i] = c.bt[p_first + i];
            c.bt = s_pages;
            c.bt_first = p_first;
        }
    }
    if (tid == kAttnWorkers) {
        s_ctx = c;
        mbar_init(bar_full, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_p, 1);
        mbar_init(bar_pv, 1);
        fence_mbar_init();
    }
    __syncthreads();
    bool ok = true;
    if (ntiles > 0) {
        // Tiles made only of keys cached before this pass do not depend on the QKV projection that precedes this
        // kernel: the first one is requested now, otherwise after the dependency has resolved.
        const bool early0 = min(c.k0 + kAttnTile, c.k1) <= base;
        if (warp == 4) {
            tmem_alloc(smem_u32(tmem_slot), tmem_cols);
            tc_fence_before();
            if (early0) attn_issue_tile<HD>(s_ctx, smem_u32(k_tile), smem_u32(v_tile), bar_full, c.k0);
        } else {
            // operands that do not depend on the predecessor: the ones, the rows' horizons and initial state
            for (int i = tid; i < SM::kOnes / 4; i += kAttnWorkers) reinterpret_cast<uint32_t*>(ones)[i] = 0x3F803F80u;
            for (int n = tid; n < kAttnMaxRows; n += kAttnWorkers) {
                const int rho = rho0 + n;
                hz[n] = n < n_rows ? base + rho % rows : -1;
                m_ref[n] = -INFINITY;
            }
        }
        pdl_wait();
        if (warp == 4) {
            if (!early0) attn_issue_tile<HD>(s_ctx, smem_u32(k_tile), smem_u32(v_tile), bar_full, c.k0);
        } else {
            // ---- stage Q (scaled by log2(e)/sqrt(hd)) as the K-major B operand, bf16 hi and lo terms:
            // piece (row n, k group g) at ((n/8) * HG + g) * 128 + (n%8) * 16
            const float scale = rsqrtf((float)HD) * 1.4426950408889634f;   // scores in the log2 domain: p = 2^(s - m)
            const int row0 = a.meta.it_row0[item];
            for (int idx = tid; idx < N * HG; idx += kAttnWorkers) {
                const int n = idx / HG, g = idx % HG;
                float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                if (n < n_rows) {
                    const int rho = rho0 + n, gq = rho / rows, r = rho % rows;
                    const float4* qp = reinterpret_cast<const float4*>(a.q + ((size_t)(row0 + r) * Hq + kvh * G + gq) * HD + g * 8);
                    const float4 x0 = qp[0], x1 = qp[1];
                    v[0] = x0.x * scale; v[1] = x0.y * scale; v[2] = x0.z * scale; v[3] = x0.w * scale;
                    v[4] = x1.x * scale; v[5] = x1.y * scale; v[6] = x1.z * scale; v[7] = x1.w * scale;
                }
                uint16_t h[8], l[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) split_bf16(v[i], h[i], l[i]);
                const uint32_t off = (uint32_t)(((n >> 3) * HG + g) * 128 + (n & 7) * 16);
                *reinterpret_cast<uint4*>(q_hi + off) = make_uint4(pack2(h[0], h[1]), pack2(h[2], h[3]), pack2(h[4], h[5]), pack2(h[6], h[7]));
                *reinterpret_cast<uint4*>(q_lo + off) = make_uint4(pack2(l[0], l[1]), pack2(l[2], l[3]), pack2(l[4], l[5]), pack2(l[6], l[7]));
            }
            fence_proxy_async_smem();      // the tensor cores read these through the asynchronous proxy
        }
        __syncthreads();                   // Q, ones and the tensor-memory base are in place
        tc_fence_after();
        const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
        const uint32_t t_S = tmem, t_O = tmem + (uint32_t)N, t_L = tmem + 2u * (uint32_t)N;

        if (warp == 4) {
            // ---------------- copies and MMA issue
            const uint32_t idesc_qk = umma_idesc_bf16(128, N, 0, 0), idesc_pv = umma_idesc_bf16(128, N, 1, 1);
            const uint32_t ka = smem_u32(k_tile), va = smem_u32(v_tile);
            const uint32_t qh = smem_u32(q_hi), ql = smem_u32(q_lo), ph = smem_u32(p_hi), pl = smem_u32(p_lo);
            const uint64_t ones_desc = umma_desc(smem_u32(ones), 2048, 128);
            for (int t = 0; t < ntiles; ++t) {
                const uint32_t par = (uint32_t)t & 1u;
                if (ok) ok = attn_wait_warp(bar_full, par);                  // K and V rows of tile t have landed
                if (lane == 0 && ok) {
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < HD / 16; ++kk)
                        umma_bf16(t_S, umma_desc(ka + kk * 256, 128, HG * 128), umma_desc(qh + kk * 256, 128, HG * 128), idesc_qk, kk > 0);
#pragma unroll
                    for (int kk = 0; kk < HD / 16; ++kk)
                        umma_bf16(t_S, umma_desc(ka + kk * 256, 128, HG * 128), umma_desc(ql + kk * 256, 128, HG * 128), idesc_qk, 1);
                    umma_commit(bar_s);
                }
                if (ok) ok = attn_wait_warp(bar_p, par);                     // P of tile t is written (and O^T rescaled)
                if (lane == 0 && ok) {
                    tc_fence_after();
                    const int n_valid = min(kAttnTile, c.k1 - (c.k0 + t * kAttnTile));
                    const int n16 = (n_valid + 15) / 16;
                    for (int ks = 0; ks < n16; ++ks) {
                        const uint64_t vd = umma_desc(va + ks * 2 * HG * 128, HG * 128, 128);
                        const uint64_t bh = umma_desc(ph + ks * 2 * NG * 128, NG * 128, 128);
                        const uint64_t bl = umma_desc(pl + ks * 2 * NG * 128, NG * 128, 128);
                        const uint32_t acc = (t > 0 || ks > 0) ? 1u : 0u;
                        umma_bf16(t_O, vd, bh, idesc_pv, acc);
                        umma_bf16(t_O, vd, bl, idesc_pv, 1);
                        umma_bf16(t_L, ones_desc, bh, idesc_pv, acc);
                        umma_bf16(t_L, ones_desc, bl, idesc_pv, 1);
                    }
                    umma_commit(bar_pv);
                }
                if (!ok) break;
                if (t + 1 < ntiles) {
                    ok = attn_wait_warp(bar_pv, par);                   // the tile's operands have been read
                    if (ok) attn_issue_tile<HD>(s_ctx, ka, va, bar_full, c.k0 + (t + 1) * kAttnTile);
                }
            }
            if (!ok && a.err && lane == 0) atomicExch(a.err, 3);
        } else {
            // ---------------- one thread per key of the tile (= tensor-memory lane)
            const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
            for (int t = 0; t < ntiles; ++t) {
                const uint32_t par = (uint32_t)t & 1u;
                const int j = c.k0 + t * kAttnTile + tid;               // this thread's key
                const int n_valid = min(kAttnTile, c.k1 - (c.k0 + t * kAttnTile));
                if (tid == 0) *s_flag = 0;
                if (ok) ok = attn_wait_warp(bar_s, par);
                tc_fence_after();
                const bool need_mask = c.k0 + (t + 1) * kAttnTile - 1 > base || n_valid < kAttnTile;   // CTA-uniform
                // ---- pass 1: the tile's maximum per row (over the 32 keys of the warp, then over the warps)
                for (int cb = 0; cb < N / 16; ++cb) {
                    float s[16];
                    tmem_ld16(t_S + lane_sel + cb * 16, s);
                    tmem_ld_wait();
                    float mine = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        float v = s[i];
                        if (need_mask && !(j < c.k1 && j <= hz[cb * 16 + i])) v = -INFINITY;
                        if (!ok) v = -INFINITY;
                        const float wmax = warp_max_redux(v);
                        if (lane == i) mine = wmax;
                    }
                    if (lane < 16) wm[warp * kAttnMaxRows + cb * 16 + lane] = mine;
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kAttnWorkers) : "memory");
                if (tid < N) {
                    const float tmax = fmaxf(fmaxf(wm[tid], wm[kAttnMaxRows + tid]), fmaxf(wm[2 * kAttnMaxRows + tid], wm[3 * kAttnMaxRows + tid]));
                    const float m_old = m_ref[tid];
                    float al = 1.f;
                    if (tmax > -INFINITY) {
                        if (m_old == -INFINITY) m_ref[tid] = tmax;             // nothing accumulated for this row so far
                        else if (tmax > m_old + kAttnLazyRescale) { m_ref[tid] = tmax; al = fast_exp2(m_old - tmax); *s_flag = 1; }
                    }
                    alpha[tid] = al;
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kAttnWorkers) : "memory");
                // the previous tile's second product has read P (and updated O^T, L): P may be overwritten
                if (t > 0 && ok) ok = attn_wait_warp(bar_pv, (uint32_t)(t - 1) & 1u);
                tc_fence_after();
                if (*s_flag && t > 0 && ok) {
                    // ---- a reference maximum moved: rescale the rows' columns of O^T and L (2N columns from t_O)
                    for (int cb = 0; cb < 2 * N / 16; ++cb) {
                        float o[16];
                        tmem_ld16(t_O + lane_sel + cb * 16, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] *= alpha[(cb * 16 + i) % N];
                        tmem_st16(t_O + lane_sel + cb * 16, o);
                    }
                    tmem_st_wait();
                }
                // ---- pass 2: p = 2^(s - reference maximum), written as the MN-major B operand (hi and lo terms):
                // piece (key group kg, row group g, key) at ((kg * NG + g) * 8 + key % 8) * 16 holds 8 rows
                for (int cb = 0; cb < N / 16; ++cb) {
                    float s[16];
                    tmem_ld16(t_S + lane_sel + cb * 16, s);
                    tmem_ld_wait();
                    uint32_t hw[8], lw[8];
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        float p2[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int n = cb * 16 + i + e;
                            const float mr = m_ref[n];
                            float v = s[i + e];
                            if (need_mask && !(j < c.k1 && j <= hz[n])) v = -INFINITY;
                            p2[e] = (ok && mr > -INFINITY) ? fast_exp2(v - mr) : 0.f;      // masked: 2^-inf = 0
                        }
                        uint16_t h0, l0, h1, l1;
                        split_bf16(p2[0], h0, l0);
                        split_bf16(p2[1], h1, l1);
                        hw[i >> 1] = pack2(h0, h1);
                        lw[i >> 1] = pack2(l0, l1);
                    }
                    const uint32_t off = (uint32_t)((((tid >> 3) * NG + cb * 2) * 8 + (tid & 7)) * 16);
                    *reinterpret_cast<uint4*>(p_hi + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                    *reinterpret_cast<uint4*>(p_hi + off + 128) = make_uint4(hw[4], hw[5], hw[6], hw[7]);
                    *reinterpret_cast<uint4*>(p_lo + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                    *reinterpret_cast<uint4*>(p_lo + off + 128) = make_uint4(lw[4], lw[5], lw[6], lw[7]);
                }
                // V rows at and beyond the split's end must be finite (P is 0 there, but 0 * NaN is not): cleared
                if (tid >= n_valid) {
#pragma unroll
                    for (int g = 0; g < HG; ++g)
                        *reinterpret_cast<uint4*>(v_tile + ((tid >> 3) * HG + g) * 128 + (tid & 7) * 16) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async_smem();
                tc_fence_before();
                asm volatile("bar.sync 1, %0;" ::"n"(kAttnWorkers) : "memory");
                if (tid == 0) mbar_arrive(bar_p);
            }
            // ---- the CTA's partial result: O^T (thread = head dimension) and L (every lane holds all rows' sums)
            if (ok) ok = attn_wait_warp(bar_pv, (uint32_t)(ntiles - 1) & 1u);
            tc_fence_after();
            for (int cb = 0; cb < N / 16; ++cb) {
                float o[16];
                tmem_ld16(t_O + lane_sel + cb * 16, o);
                tmem_ld_wait();
                if (tid < HD) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) Fo[(size_t)(cb * 16 + i) * HD + tid] = ok ? o[i] : 0.f;
                }
            }
            for (int cb = 0; cb < N / 16; ++cb) {       // thread n keeps row n's sum (its own lane's copy)
                float l[16];
                tmem_ld16(t_L + lane_sel + cb * 16, l);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    if (tid == cb * 16 + i) Fl[tid] = ok ? l[i] : 0.f;
            }
            if (!ok && a.err && lane == 0) atomicExch(a.err, 4);
            tc_fence_before();
        }
        __syncthreads();
        if (warp == 4) {
            tc_fence_after();
            tmem_dealloc(tmem, tmem_cols);
        }
    } else {
        // empty split: contributes nothing (finite zeros, so the merge can read it unconditionally)
        pdl_wait();
        for (int i = tid; i < N; i += kAttnThreads) { Fm[i] = -INFINITY; Fl[i] = 0.f; }
        for (int i = tid; i < N * HD; i += kAttnThreads) Fo[i] = 0.f;
    }

    // ---- merge the cluster's splits over distributed shared memory; rank r owns rows r, r+cs, ... of the group
    cluster_sync_all();
    constexpr int EPT = HD / kAttnWorkers > 0 ? HD / kAttnWorkers : 1;   // output columns per thread
    const uint32_t fo_a = smem_u32(Fo), fm_a = smem_u32(Fm), fl_a = smem_u32(Fl);
    const int row0 = a.meta.it_row0[item];
    const int KSo = (Hq * HD) / 16, NTo = xf_nt(a.M);
    const size_t slot0 = (size_t)a.meta.it_part0[item] + ((size_t)kvh * R + rho0) * ncl;   // + rl*ncl + cluster
#pragma unroll 2
    for (int rl = rank; rl < n_rows; rl += cs) {
        // all remote reads of a row are issued together: cs maxima, cs sums, cs output values per thread
        float ms[kAttnMaxCluster], ls[kAttnMaxCluster], ov[EPT][kAttnMaxCluster];
#pragma unroll
        for (int r = 0; r < kAttnMaxCluster; ++r) {
            if (r >= cs) {                       // beyond this launch's cluster: an empty split
                ms[r] = -INFINITY; ls[r] = 0.f;
#pragma unroll
                for (int k = 0; k < EPT; ++k) ov[k][r] = 0.f;
                continue;
            }
            ms[r] = dsmem_ld_f32(dsmem_addr(fm_a + rl * 4, (uint32_t)r));
            ls[r] = dsmem_ld_f32(dsmem_addr(fl_a + rl * 4, (uint32_t)r));
#pragma unroll
            for (int k = 0; k < EPT; ++k) {
                const int e = tid + k * kAttnWorkers;
                ov[k][r] = (e < HD && tid < kAttnWorkers) ? dsmem_ld_f32(dsmem_addr(fo_a + (uint32_t)(rl * HD + e) * 4, (uint32_t)r)) : 0.f;
            }
        }
        float m = -INFINITY;
#pragma unroll
        for (int r = 0; r < kAttnMaxCluster; ++r) m = fmaxf(m, ms[r]);
        float den = 0.f, w[kAttnMaxCluster];
#pragma unroll
        for (int r = 0; r < kAttnMaxCluster; ++r) {
            w[r] = (ms[r] == -INFINITY) ? 0.f : exp2f(ms[r] - m);   // an empty split or one beyond the causal horizon
            den += w[r] * ls[r];
        }
        const int rho = rho0 + rl, gq = rho / rows, r_in = rho % rows;
#pragma unroll
        for (int k = 0; k < EPT; ++k) {
            const int e = tid + k * kAttnWorkers;
            if (e < HD && tid < kAttnWorkers) {
                float num = 0.f;
#pragma unroll
                for (int r = 0; r < kAttnMaxCluster; ++r) num += w[r] * ov[k][r];
                if (ncl == 1) xf_store_one(a.xf_out, row0 + r_in, (kvh * G + gq) * HD + e, num / den, KSo, NTo);
                else a.o_part[(slot0 + (size_t)rl * ncl + cl) * HD + e] = num;     // un-normalised, with (m, den)
            }
        }
        if (ncl > 1 && tid == 0) {
            a.m_part[slot0 + (size_t)rl * ncl + cl] = m;
            a.l_part[slot0 + (size_t)rl * ncl + cl] = den;
        }
    }
    if (ncl > 1) __threadfence();
    cluster_sync_all();   // nobody leaves while its shared memory may still be read; partials are published
    if (ncl == 1) return;
    // ---- several clusters share the keys: the last one to arrive merges their partials
    if (rank == 0 && tid == 0) {
        int* ticket = a.tickets + ((size_t)item * Hkv + kvh) * a.row_groups + rg;
        const int t = atomicAdd(ticket, 1);
        const int last = (t == ncl - 1);
        if (last) *ticket = 0;                                   // self-cleaning: ready for the next launch
        const uint32_t fa = smem_u32(s_last);
        for (int r = 0; r < cs; ++r) dsmem_st_f32(dsmem_addr(fa, (uint32_t)r), __int_as_float(last));
    }
    cluster_sync_all();
    if (!*s_last) return;
    __threadfence();
    for (int rl = rank; rl < n_rows; rl += cs) {
        float ms[kMaxSplits / kAttnSplits], ls[kMaxSplits / kAttnSplits], ov[EPT][kMaxSplits / kAttnSplits];
#pragma unroll
        for (int j = 0; j < kMaxSplits / kAttnSplits; ++j) {
            const bool on = j < ncl;
            const size_t sl = slot0 + (size_t)rl * ncl + j;
            ms[j] = on ? __ldcg(a.m_part + sl) : -INFINITY;
            ls[j] = on ? __ldcg(a.l_part + sl) : 0.f;
#pragma unroll
            for (int k = 0; k < EPT; ++k) {
                const int e = tid + k * kAttnWorkers;
                ov[k][j] = (on && e < HD && tid < kAttnWorkers) ? __ldcg(a.o_part + sl * HD + e) : 0.f;
            }
        }
        float m = -INFINITY;
#pragma unroll
        for (int j = 0; j < kMaxSplits / kAttnSplits; ++j) m = fmaxf(m, ms[j]);
        float den = 0.f, w[kMaxSplits / kAttnSplits];
#pragma unroll
        for (int j = 0; j < kMaxSplits / kAttnSplits; ++j) {
            w[j] = (ms[j] == -INFINITY) ? 0.f : exp2f(ms[j] - m);
            den += w[j] * ls[j];
        }
        const int rho = rho0 + rl, gq = rho / rows, r_in = rho % rows;
#pragma unroll
        for (int k = 0; k < EPT; ++k) {
            const int e = tid + k * kAttnWorkers;
            if (e < HD && tid < kAttnWorkers) {
                float num = 0.f;
#pragma unroll
                for (int j = 0; j < kMaxSplits / kAttnSplits; ++j) num += w[j] * ov[k][j];
                xf_store_one(a.xf_out, row0 + r_in, (kvh * G + gq) * HD + e, num / den, KSo, NTo);
            }
        }
    }
}

}  // namespace pipesd
