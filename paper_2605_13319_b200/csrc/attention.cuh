// Multi-query decode attention over a paged bf16 KV cache on the tcgen05 tensor cores: each request contributes a
// short chunk of query rows (the pending token plus its k drafts) that attend to the cached prefix and, causally,
// to each other.  The keys of a request are cut into up to 16 splits ("split-K"), one CTA each; a CTA leaves an
// un-normalised partial output with its reference maximum and sum in global memory (a few MB that stay in L2),
// takes a ticket, and the last CTA of a (request, KV head, row group) to arrive merges the splits in split order
// and writes the result straight into the output projection's input format -- nobody waits for anybody, and a CTA
// that is not the last one leaves its SM to the next kernel at once.
//
// One CTA = one KV head of one request x one key split x up to 112 query rows, where the rows are all (query head
// of the group, chunk row) pairs that share the KV head (GQA).  The keys are on the M side of the MMAs, the (few)
// query rows on the narrow N side:
//   S^T[128 keys x N rows] = K_tile[128 x hd] . Q^T[hd x N]          A = K rows from the cache, B = Q
//   O^T[hd x N rows]      += V_tile^T[hd x 128 keys] . P^T[128 x N]   A = V rows from the cache, B = P
//   L  [  * x N rows]      += 1[* x 128 keys] . P^T[128 x N]          the softmax denominators, by the same P
// with S^T (twice: two tiles in flight), O^T and L in tensor memory (4N columns).  The cache stores, per page and
// head, the rows in 8-row groups of 8-element pieces ([slot/8][hd/8][slot%8][8]), which IS the operand order of
// both products (K-major for the first, MN-major for the second): a page lands in shared memory by one bulk copy
// and is read by the tensor cores as it is.  Q and P are fp32 values split into bf16 hi + lo terms (two MMAs into
// the same accumulator); K and V are the cache's bf16.
// Warps 0-7: one thread per key of a tile (= tensor-memory lane; warps w and w+4 share a lane quarter and take
// alternate 16-row column blocks): masking, the running maximum (a row's reference maximum only moves when the
// tile's maximum exceeds it by more than 2^8, so that O^T is rarely rescaled), exponentials, P written back as the
// next MMA's B operand.  Warp 8: bulk copies of the K/V pages (a ring of three slots, K0 V0 K1 V1 ...; tiles of keys
// that were cached before this pass do not depend on the preceding QKV projection and are requested before the
// dependent-launch wait) and the MMA issue (one thread).  Every wait is bounded and raises the device error word.
#pragma once
#include "common.cuh"
#include "layers.cuh"
#include "tcgen05.cuh"

namespace pipesd {

constexpr int kAttnWorkers = 256;           // threads of warps 0-7
constexpr int kAttnThreads = kAttnWorkers + 32;
constexpr int kAttnTile = 128;              // keys per tile = M of the MMAs
constexpr int kAttnMaxRows = 112;           // query rows per CTA (N of the MMAs; what fits beside the ring); more rows: more row groups
constexpr int kAttnMaxSplits = 16;          // key splits of one request
constexpr int kAttnShortTail = 112;         // keys of the second tile up to which the third ring slot is cut down
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

// Shared-memory plan of one CTA with N query rows (a multiple of 16).  K and V tiles travel through a ring of three
// slots in the order K0 V0 K1 V1 ...: two of a whole tile each and a third of `slot_c` bytes (a whole tile, or less
// when no CTA of the launch has more than two tiles, the second of at most kAttnShortTail keys: the K/V of such a
// CTA are then requested in full before the first product starts).
template <int HD>
struct AttnSmem {
    static constexpr int kTileBytes = kAttnTile * HD * 2;            // one K or V tile
    static constexpr int kOnes = 256;                                 // 16 keys x 8 ones: the denominators' A operand
    __host__ __device__ static constexpr int q_bytes(int N) { return N * HD * 2; }          // hi or lo
    __host__ __device__ static constexpr int p_bytes(int N) { return kAttnTile * N * 2; }   // hi or lo
    __host__ __device__ static constexpr int small_bytes(int N) { return 8 * N * 4 + 128; } // warp maxima [4][N], horizon, reference
                                                                                            // maximum, factor, sums [N] each; barriers
    __host__ __device__ static constexpr size_t bytes(int N, int slot_c) {
        return (size_t)kOnes + 2 * kTileBytes + slot_c + 2 * q_bytes(N) + 2 * p_bytes(N) + small_bytes(N);
    }
};

// Tensor-memory columns of a CTA with N query rows: S^T twice, O^T and L, N columns each, as a power of two >= 32.
__host__ __device__ constexpr int attn_tmem_cols(int N) {
    int c = 32;
    while (c < 4 * N) c *= 2;
    return c;
}
static inline int attn_slot_c_bytes(int hd, bool short_tail) { return (short_tail ? kAttnShortTail : kAttnTile) * hd * 2; }
// Dynamic shared memory to ask for: the plan above, padded so that the CTAs an SM can hold never want more than the
// SM's 512 tensor-memory columns together (the allocation instruction blocks until its columns are free).
static inline size_t attn_smem_bytes(int hd, int N, bool short_tail) {
    const int sc = attn_slot_c_bytes(hd, short_tail);
    const size_t need = hd == 128 ? AttnSmem<128>::bytes(N, sc) : AttnSmem<64>::bytes(N, sc);
    const int max_ctas = 512 / attn_tmem_cols(N);
    const size_t floor_ = (size_t)(227 * 1024) / (max_ctas + 1) + 1;
    return need > floor_ ? need : floor_;
}
static inline int attn_rows_n(int rows_per_kv_head) {    // N of a CTA that holds this many query rows
    const int r = rows_per_kv_head > kAttnMaxRows ? kAttnMaxRows : rows_per_kv_head;
    return (r + 15) / 16 * 16;
}

// Host: how one request's keys are split.  `units` = CTA groups that compete for the device per layer, counted in
// groups of this request's length: for a request verified alone its KV heads x row groups; in a batch the batch's
// (keys x groups) total divided by this request's keys.  slots[0 | 1] = CTAs of this kernel the device keeps resident
// at once for the request's row count with the whole | cut-down third ring slot.  As many splits as let all CTAs of the
// pass run in one wave (at most 16, at most one per 128 keys), then the fewest splits that leave each CTA the same
// number of 128-key tiles.  The plan fixes the order a row's keys are summed in: a function of the pass's composition
// and the device, the same every time that composition is verified.
struct AttnSplit { int splits, keys_per_split, short_tail; };
static inline AttnSplit attn_split_plan(int total_keys, int page_size, int units, const int* slots) {
    auto chunk_of = [&](int s) {
        const int ch = (total_keys + s - 1) / s;
        return (ch + page_size - 1) / page_size * page_size;
    };
    auto tiles_of = [&](int s) { return (chunk_of(s) + kAttnTile - 1) / kAttnTile; };
    const int by_keys = (total_keys + kAttnTile - 1) / kAttnTile;
    AttnSplit p = {1, chunk_of(1), 0};
    for (int cls = 1; cls >= 0; --cls) {
        int s = slots[cls] / (units > 0 ? units : 1);
        s = s > kAttnMaxSplits ? kAttnMaxSplits : s;
        s = s > by_keys ? by_keys : s;
        s = s < 1 ? 1 : s;
        const int t = tiles_of(s);
        while (s > 1 && tiles_of(s - 1) == t) --s;
        p.splits = s;
        p.keys_per_split = chunk_of(s);
        p.short_tail = cls;
        if (cls == 0 || p.keys_per_split <= kAttnTile + kAttnShortTail) break;
    }
    return p;
}

// Per-CTA constants of the tile copies.
struct AttnCtx {
    const uint16_t* kbase;     // K block of page 0 for this layer and KV head
    const int32_t* bt;         // page ids of the request
    size_t page_stride;        // elements between consecutive pages of a layer
    size_t v_off;              // elements from a K block to the V block of the same page and head
    int page_size;
    int k0, k1;
};

// Issue (one warp) the copies of the K rows (kv = 0) or V rows (kv = 1) of one 128-key tile: the rows of a page that
// belong to one KV head are contiguous in the pool, already in operand order, so every page the tile touches is one
// bulk copy (lane l takes the l-th page), counted in bytes on the barrier.  Whole 8-row groups are copied: the rows
// of the last group at or beyond k1 are masked (K) or cleared (V) by the consumers.
template <int HD>
__device__ __forceinline__ void attn_issue_tile(const AttnCtx& c, int kv, uint32_t dst, uint32_t bar, int j0) {
    const int lane = threadIdx.x & 31;
    const int j1 = (min(j0 + kAttnTile, c.k1) + 7) & ~7;
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)(j1 - j0) * (HD * 2));
    __syncwarp();
    const int pidx = j0 / c.page_size + lane;                              // page of the request
    const int js = max(j0, pidx * c.page_size), je = min(j1, (pidx + 1) * c.page_size);
    if (js < je) {
        const uint16_t* src = c.kbase + (size_t)c.bt[pidx] * c.page_stride + (kv ? c.v_off : 0) +
                              (size_t)(js - pidx * c.page_size) * HD;
        bulk_g2s(dst + (uint32_t)(js - j0) * (HD * 2), src, (uint32_t)(je - js) * (HD * 2), bar);
    }
}

struct AttnArgs {
    const float* q;            // [M][Hq*hd] rotated queries
    PassMeta meta;
    const uint16_t* kv_pool;
    int layer, n_pages, page_size, M, Hq, Hkv;
    int rows_cap;              // query rows per row group (kAttnMaxRows, or 16 for a batch whose requests have up to 32)
    int n_max;                 // N the launch's shared memory was sized for
    int slot_c;                // bytes of the ring's third slot
    int row_groups;
    float* o_part;             // partial results: [slot][hd], slot = it_part0 + ((kv head * R + row) * splits + split)
    float* m_part;             // [slot]
    float* l_part;             // [slot]
    int* tickets;              // [item][kv head][row group], zero between launches
    uint16_t* xf_out;          // the output projection's input: split-bf16 fragments, or (xd_tbs > 0) an xd array
    int xd_tbs;
    // Weights of the projections that follow (nullable): while this kernel runs, HBM carries little besides the K/V
    // it reads.  Once a CTA's own K/V tiles have all landed, its copy warp asks the L2 for this CTA's share of the
    // first pf_len[i] bytes at pf_ptr[i] (128-byte lines dealt over the whole grid).  Purely a hint.
    const unsigned char* pf_ptr[2];
    size_t pf_len[2];
    int* err;
};

// grid (max splits of the launch, n_kv_heads * row_groups, n_items), block 288.  The register bound is what lets two CTAs
// share an SM: a CTA's nine warps put three on one of the SM's four register partitions (16K registers each), and two
// such triples must fit it.
template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 3) attn_kernel(const AttnArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    using SM = AttnSmem<HD>;
    constexpr int HG = HD / 8;                                      // 8-element pieces of a row
    pdl_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int item = a.meta.it_order[blockIdx.z];
    // per-request constants: independent loads, in flight together
    const int nsplit = a.meta.it_nsplit[item];
    const int rows = a.meta.it_rows[item];
    const int base = a.meta.it_base[item];
    const int chunk = a.meta.it_chunk[item];
    const int row0 = a.meta.it_row0[item];
    const int part0 = a.meta.it_part0[item];
    const int req_slot = a.meta.it_slot[item];
    const int sp = blockIdx.x;                                     // key split of this CTA
    if (sp >= nsplit) return;
    const int Hkv = a.Hkv, Hq = a.Hq;
    const int kvh = blockIdx.y % Hkv, rg = blockIdx.y / Hkv;
    const int G = Hq / Hkv;
    const int R = G * rows;
    const int rho0 = rg * a.rows_cap;
    if (rho0 >= R) return;
    const int n_rows = min(a.rows_cap, R - rho0);
    const int N = (n_rows + 15) & ~15;
    if (N > a.n_max) return;
    const int NG = N / 8, NB = N / 16;
    const int total = base + rows;
    AttnCtx c;
    c.k0 = min(sp * chunk, total);
    c.k1 = min(c.k0 + chunk, total);
    c.kbase = a.kv_pool + kv_index(a.layer, a.n_pages, 0, 0, Hkv, kvh, a.page_size, 0, HD, 0);
    c.page_stride = (size_t)2 * Hkv * a.page_size * HD;
    c.v_off = (size_t)Hkv * a.page_size * HD;
    c.page_size = a.page_size;
    c.bt = a.meta.block_tab + (size_t)req_slot * a.meta.max_pages;
    const int ntiles = c.k1 > c.k0 ? (c.k1 - c.k0 + kAttnTile - 1) / kAttnTile : 0;
    const size_t slot0 = (size_t)part0 + ((size_t)kvh * R + rho0) * nsplit;     // + row * nsplit + split
    const int KSo = (Hq * HD) / 16, NTo = xf_nt(a.M);

    // ---- shared memory: the ones come first (the tensor cores read a few KB past them, see below)
    unsigned char* ones = smem;
    unsigned char* ring = ones + SM::kOnes;                        // slots 0, 1: a whole tile; slot 2: a.slot_c bytes
    unsigned char* q_hi = ring + 2 * SM::kTileBytes + a.slot_c;
    unsigned char* q_lo = q_hi + SM::q_bytes(N);
    unsigned char* p_hi = q_lo + SM::q_bytes(N);
    unsigned char* p_lo = p_hi + SM::p_bytes(N);
    float* wm = reinterpret_cast<float*>(p_lo + SM::p_bytes(N));   // [4][N] maxima of a tile per lane quarter
    int* hz = reinterpret_cast<int*>(wm + 4 * N);                  // [N] last visible key of a row (-1: padding row)
    float* m_ref = reinterpret_cast<float*>(hz + N);               // [N] reference maximum of a row
    float* alpha = m_ref + N;                                      // [N] rescale factor of a row for this tile
    float* Fl = alpha + N;                                         // [N] the CTA's partial denominators
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(Fl + N);   // full[3], s_full[2], p_full, pv_done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 7);
    int* s_flag = reinterpret_cast<int*>(tmem_slot + 1);           // a row's reference maximum moved: rescale
    int* s_last = s_flag + 1;
    const uint32_t bar_full = smem_u32(bars), bar_s = bar_full + 24, bar_p = bar_full + 40, bar_pv = bar_full + 48;
    const uint32_t tmem_cols = (uint32_t)attn_tmem_cols(N);
    const uint32_t ring_a = smem_u32(ring);
    auto slot_addr = [&](int i) { return ring_a + (uint32_t)(i % 3) * SM::kTileBytes; };   // ring slot of item i (K_t: 2t, V_t: 2t+1)

    bool ok = true;
    uint32_t tmem_held = 0;        // tensor memory to give back before leaving, if any (address 0 is a valid one)
    bool holds_tmem = false;
    // Tensor memory is released off the critical path: after the partial result has been announced.
    auto release_tmem = [&]() {
        if (holds_tmem && warp == 8) {
            tc_fence_after();
            tmem_dealloc(tmem_held, tmem_cols);
        }
    };
    if (ntiles > 0) {
        uint32_t tmem = 0;
        if (warp == 8) {
            // ---------------- barriers, the first three items of the ring, tensor memory
            if (lane == 0) {
                for (int i = 0; i < 7; ++i) mbar_init(bar_full + 8 * i, 1);
                fence_mbar_init();
            }
            __syncwarp();
            // Items made only of keys cached before this pass do not depend on the QKV projection that precedes this
            // kernel: they are requested now, the others after the dependency has resolved.
            const int early_tiles = base >= c.k1 ? ntiles : (base - c.k0) / kAttnTile;      // whole tiles below `base`
            const int first = ntiles > 1 ? 3 : 2;                                            // items requested up front
            for (int i = 0; i < first; ++i)
                if ((i >> 1) < early_tiles) attn_issue_tile<HD>(c, i & 1, slot_addr(i), bar_full + 8 * (i % 3), c.k0 + (i >> 1) * kAttnTile);
            tmem_alloc(smem_u32(tmem_slot), tmem_cols);
            tc_fence_before();
            pdl_wait();
            for (int i = 0; i < first; ++i)
                if ((i >> 1) >= early_tiles) attn_issue_tile<HD>(c, i & 1, slot_addr(i), bar_full + 8 * (i % 3), c.k0 + (i >> 1) * kAttnTile);
        } else {
            // operands that do not depend on the predecessor: the ones, the rows' horizons and initial state
            if (tid < SM::kOnes / 4) reinterpret_cast<uint32_t*>(ones)[tid] = 0x3F803F80u;
            for (int n = tid; n < N; n += kAttnWorkers) {
                const int rho = rho0 + n;
                hz[n] = n < n_rows ? base + rho % rows : -1;
                m_ref[n] = -INFINITY;
            }
            pdl_wait();
            // ---- stage Q (scaled by log2(e)/sqrt(hd)) as the K-major B operand, bf16 hi and lo terms:
            // piece (row n, k group g) at ((n/8) * HG + g) * 128 + (n%8) * 16.  Two pieces per thread and step, all
            // loads of a step in flight together.
            const float scale = rsqrtf((float)HD) * 1.4426950408889634f;   // scores in the log2 domain: p = 2^(s - m)
            for (int idx0 = tid; idx0 < N * HG; idx0 += 2 * kAttnWorkers) {
                float4 x[2][2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int idx = idx0 + u * kAttnWorkers, n = idx / HG, g = idx % HG;
                    x[u][0] = x[u][1] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (idx < N * HG && n < n_rows) {
                        const int rho = rho0 + n, gq = rho / rows, r = rho % rows;
                        const float4* qp = reinterpret_cast<const float4*>(a.q + ((size_t)(row0 + r) * Hq + kvh * G + gq) * HD + g * 8);
                        x[u][0] = qp[0];
                        x[u][1] = qp[1];
                    }
                }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int idx = idx0 + u * kAttnWorkers, n = idx / HG, g = idx % HG;
                    if (idx >= N * HG) break;
                    const float v[8] = {x[u][0].x * scale, x[u][0].y * scale, x[u][0].z * scale, x[u][0].w * scale,
                                        x[u][1].x * scale, x[u][1].y * scale, x[u][1].z * scale, x[u][1].w * scale};
                    uint16_t h[8], l[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) split_bf16(v[i], h[i], l[i]);
                    const uint32_t off = (uint32_t)(((n >> 3) * HG + g) * 128 + (n & 7) * 16);
                    *reinterpret_cast<uint4*>(q_hi + off) = make_uint4(pack2(h[0], h[1]), pack2(h[2], h[3]), pack2(h[4], h[5]), pack2(h[6], h[7]));
                    *reinterpret_cast<uint4*>(q_lo + off) = make_uint4(pack2(l[0], l[1]), pack2(l[2], l[3]), pack2(l[4], l[5]), pack2(l[6], l[7]));
                }
            }
            fence_proxy_async_smem();      // the tensor cores read these through the asynchronous proxy
        }
        __syncthreads();                   // barriers, Q, ones and the tensor-memory base are in place
        tc_fence_after();
        tmem = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
        const uint32_t t_S = tmem, t_O = tmem + 2u * (uint32_t)N, t_L = tmem + 3u * (uint32_t)N;   // S^T twice, O^T, L

        if (warp == 8) {
            // ---------------- copies and MMA issue.  Ring item i (K_t: 2t, V_t: 2t+1) lives in slot i % 3 and may be
            // requested once item i - 3 has been read: a K tile by the first product of its tile (s_full), a V tile by
            // the second (pv_done).  The first product of tile t+1 is issued ahead of the second of tile t.
            const uint32_t idesc_qk = umma_idesc_bf16(128, N, 0, 0), idesc_pv = umma_idesc_bf16(128, N, 1, 1);
            const uint32_t qh = smem_u32(q_hi), ql = smem_u32(q_lo), ph = smem_u32(p_hi), pl = smem_u32(p_lo);
            // the denominators' A operand: 16 keys x 8 rows of ones; the other 120 rows of the MMA read whatever follows
            // in shared memory (the ring) and land in tensor-memory lanes that nobody reads
            const uint64_t ones_desc = umma_desc(smem_u32(ones), 128, 256);
            auto issue_qk = [&](int t) {       // S^T[t & 1] = K_t . Q^T
                const uint32_t ka = slot_addr(2 * t), d = t_S + (uint32_t)((t & 1) * N);
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk)
                    umma_bf16(d, umma_desc(ka + kk * 256, 128, HG * 128), umma_desc(qh + kk * 256, 128, HG * 128), idesc_qk, kk > 0);
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk)
                    umma_bf16(d, umma_desc(ka + kk * 256, 128, HG * 128), umma_desc(ql + kk * 256, 128, HG * 128), idesc_qk, 1);
                umma_commit(bar_s + 8 * (t & 1));
            };
            auto full_wait = [&](int i) { return attn_wait_warp(bar_full + 8 * (i % 3), (uint32_t)(i / 3) & 1u); };
            auto request = [&](int i) {        // ring item i, if the split has it
                if ((i >> 1) < ntiles) attn_issue_tile<HD>(c, i & 1, slot_addr(i), bar_full + 8 * (i % 3), c.k0 + (i >> 1) * kAttnTile);
            };
            ok = full_wait(0);
            if (ok && lane == 0) { tc_fence_after(); issue_qk(0); }
            for (int t = 0; t < ntiles && ok; ++t) {
                if (t + 1 < ntiles) {
                    ok = full_wait(2 * t + 2);                                           // K of tile t+1 has landed
                    // S^T[(t+1) & 1] was last read for tile t-1: free once P of tile t-1 was announced (seen below)
                    if (ok && lane == 0) { tc_fence_after(); issue_qk(t + 1); }
                }
                if (ok) ok = attn_wait_warp(bar_s + 8 * (t & 1), (uint32_t)(t >> 1) & 1u);   // K_t has been read
                if (ok && t + 1 < ntiles) request(2 * t + 3);                            // V of tile t+1 into K_t's slot
                if (ok) ok = attn_wait_warp(bar_p, (uint32_t)t & 1u);                    // P of tile t is written (and O^T rescaled)
                if (ok) ok = full_wait(2 * t + 1);                                       // V of tile t has landed
                if (ok && lane == 0) {
                    tc_fence_after();
                    const uint32_t va = slot_addr(2 * t + 1);
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
                if (ok && t == ntiles - 1) {
                    // every K/V tile of this CTA has landed and its last products are issued: hints for the weights
                    // of the projections that follow
                    const size_t n_thr = (size_t)gridDim.x * gridDim.y * gridDim.z * 32;
                    const size_t g = (((size_t)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * 32 + lane;
#pragma unroll
                    for (int r = 0; r < 2; ++r)
                        if (a.pf_ptr[r] != nullptr)
                            for (size_t o = g * 128; o < a.pf_len[r]; o += n_thr * 128)
                                asm volatile("prefetch.global.L2 [%0];" ::"l"(a.pf_ptr[r] + o) : "memory");
                }
                if (ok && t + 2 < ntiles) {
                    ok = attn_wait_warp(bar_pv, (uint32_t)t & 1u);                       // V_t has been read
                    if (ok) request(2 * t + 4);                                          // K of tile t+2 into V_t's slot
                }
            }
            if (!ok && a.err && lane == 0) atomicExch(a.err, 3);
        } else {
            // ---------------- thread = key of the tile (tensor-memory lane 32 * quarter + lane); the two warps of a
            // lane quarter take alternate 16-row column blocks
            const int quarter = warp & 3, half = warp >> 2;
            const int kt = quarter * 32 + lane;                         // key within the tile
            const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
            for (int t = 0; t < ntiles; ++t) {
                const int j = c.k0 + t * kAttnTile + kt;                // this thread's key
                const int n_valid = min(kAttnTile, c.k1 - (c.k0 + t * kAttnTile));
                const uint32_t t_St = t_S + (uint32_t)((t & 1) * N);
                if (tid == 0) *s_flag = 0;
                if (ok) ok = attn_wait_warp(bar_s + 8 * (t & 1), (uint32_t)(t >> 1) & 1u);
                tc_fence_after();
                const bool need_mask = c.k0 + (t + 1) * kAttnTile - 1 > base || n_valid < kAttnTile;   // CTA-uniform
                // ---- pass 1: the tile's maximum per row (over the 32 keys of the warp, then over the lane quarters)
                for (int cu = half; cu < NG; cu += 2) {
                    float s[8];
                    tmem_ld8(t_St + lane_sel + cu * 8, s);
                    tmem_ld_wait();
                    float mine = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float v = s[i];
                        if (need_mask && !(j < c.k1 && j <= hz[cu * 8 + i])) v = -INFINITY;
                        if (!ok) v = -INFINITY;
                        const float wmax = warp_max_redux(v);
                        if (lane == i) mine = wmax;
                    }
                    if (lane < 8) wm[quarter * N + cu * 8 + lane] = mine;
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kAttnWorkers) : "memory");
                if (tid < N) {
                    const float tmax = fmaxf(fmaxf(wm[tid], wm[N + tid]), fmaxf(wm[2 * N + tid], wm[3 * N + tid]));
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
                    for (int cb = half; cb < 2 * NB; cb += 2) {
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
                for (int cu = half; cu < NG; cu += 2) {
                    float s[8];
                    tmem_ld8(t_St + lane_sel + cu * 8, s);
                    tmem_ld_wait();
                    uint32_t hw[4], lw[4];
#pragma unroll
                    for (int i = 0; i < 8; i += 2) {
                        float p2[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int n = cu * 8 + i + e;
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
                    const uint32_t off = (uint32_t)((((kt >> 3) * NG + cu) * 8 + (kt & 7)) * 16);
                    *reinterpret_cast<uint4*>(p_hi + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                    *reinterpret_cast<uint4*>(p_lo + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                }
                // V rows at and beyond the split's end must be finite (P is 0 there, but 0 * NaN is not): cleared, once
                // the tile's V rows have landed (the copy may bring garbage rows of the last 8-row group)
                if (n_valid < kAttnTile) {
                    if (ok) ok = attn_wait_warp(bar_full + 8 * ((2 * t + 1) % 3), (uint32_t)((2 * t + 1) / 3) & 1u);
                    if (half == 0 && kt >= n_valid && kt < ((n_valid + 15) & ~15)) {
                        unsigned char* v_tile = ring + ((2 * t + 1) % 3) * SM::kTileBytes;
#pragma unroll
                        for (int g = 0; g < HG; ++g)
                            *reinterpret_cast<uint4*>(v_tile + ((kt >> 3) * HG + g) * 128 + (kt & 7) * 16) = make_uint4(0, 0, 0, 0);
                    }
                }
                fence_proxy_async_smem();
                tc_fence_before();
                asm volatile("bar.sync 1, %0;" ::"n"(kAttnWorkers) : "memory");
                if (tid == 0) mbar_arrive(bar_p);
            }
            // ---- the CTA's partial result: O^T (thread = head dimension) and L (lanes 0-7 hold all rows' sums)
            if (ok) ok = attn_wait_warp(bar_pv, (uint32_t)(ntiles - 1) & 1u);
            tc_fence_after();
            if (quarter == 0) {
                // the column blocks go to the two warps of the quarter the other way round than O^T's below, so that with
                // one block the denominators are stored by a warp that has no O^T columns to store
                for (int cb = half ^ 1; cb < NB; cb += 2) {
                    float l[16];
                    tmem_ld16(t_L + cb * 16, l);
                    tmem_ld_wait();
                    if (lane == 0) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) Fl[cb * 16 + i] = ok ? l[i] : 0.f;
                    }
                    __syncwarp();
                    const int n = cb * 16 + lane;
                    if (nsplit > 1 && lane < 16 && n < n_rows) {         // lane = row: one store each
                        a.l_part[slot0 + (size_t)n * nsplit + sp] = Fl[n];
                        a.m_part[slot0 + (size_t)n * nsplit + sp] = m_ref[n];
                    }
                }
            }
            // nothing to merge: the rows are normalised and stored as the output projection's input.  Where a row lands
            // there (its token, its head's first k16 step) is worked out once per row, into the maxima's array
            uint32_t* otab = reinterpret_cast<uint32_t*>(wm);
            if (nsplit == 1 && tid < n_rows) {
                const int rho = rho0 + tid, gq = rho / rows, r_in = rho % rows;
                otab[tid] = act_index_row(row0 + r_in, ((kvh * G + gq) * HD) >> 4, KSo, NTo, a.xd_tbs);
            }
            const uint32_t ocol = act_index_col(kt, NTo, a.xd_tbs), olo = act_index_lo(a.xd_tbs);
            if (nsplit == 1) asm volatile("bar.sync 1, %0;" ::"n"(kAttnWorkers) : "memory");     // the sums and the table
            for (int cb = half; cb < NB; cb += 2) {
                float o[16];
                tmem_ld16(t_O + lane_sel + cb * 16, o);
                tmem_ld_wait();
                if (kt < HD) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int n = cb * 16 + i;
                        if (n < n_rows) {
                            const float v = ok ? o[i] : 0.f;
                            if (nsplit == 1) {
                                act_store_at(a.xf_out, otab[n] + ocol, olo, v / Fl[n]);
                            } else {
                                a.o_part[(slot0 + (size_t)n * nsplit + sp) * HD + kt] = v;
                            }
                        }
                    }
                }
            }
            if (!ok && a.err && lane == 0) atomicExch(a.err, 4);
            tc_fence_before();
        }
        __syncthreads();
        tmem_held = tmem;
        holds_tmem = true;
    } else {
        // empty split: contributes nothing (finite zeros, so the merge can read it unconditionally)
        pdl_wait();
        for (int i = tid; i < n_rows * HD; i += kAttnThreads) a.o_part[(slot0 + (size_t)(i / HD) * nsplit + sp) * HD + i % HD] = 0.f;
        for (int i = tid; i < n_rows; i += kAttnThreads) {
            a.m_part[slot0 + (size_t)i * nsplit + sp] = -INFINITY;
            a.l_part[slot0 + (size_t)i * nsplit + sp] = 0.f;
        }
        __syncthreads();
    }
    if (nsplit == 1) { release_tmem(); return; }

    // ---- the last CTA of this (request, KV head, row group) to arrive merges the splits, in split order
    // (the barrier above orders the whole CTA's stores before thread 0's ticket, a release; the ticket is also an acquire,
    // and the barrier below orders it before everybody's loads of the other CTAs' partials)
    if (tid == 0) {
        int* ticket = a.tickets + ((size_t)item * Hkv + kvh) * a.row_groups + rg;
        int t;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(t) : "l"(ticket) : "memory");
        const int last = (t == nsplit - 1);
        if (last) *ticket = 0;                                   // self-cleaning: ready for the next launch
        *s_last = last;
    }
    __syncthreads();
    release_tmem();
    if (!*s_last) return;
    // warp = row, lane = four columns: one round covers nine rows.  All of a row's loads are issued before the first
    // use (one trip to the L2 for up to kMergeBatch splits): lane j fetches split j's maximum and denominator, every
    // lane its four columns of each split's numerator; the sums run in split order.
    constexpr int kMergeBatch = 10;
    for (int rl = warp; rl < n_rows; rl += kAttnThreads / 32) {
        const size_t sl0 = slot0 + (size_t)rl * nsplit;
        const float m_mine = lane < nsplit ? __ldcg(a.m_part + sl0 + lane) : -INFINITY;
        const float l_mine = lane < nsplit ? __ldcg(a.l_part + sl0 + lane) : 0.f;
        float4 ov[kMergeBatch];
#pragma unroll
        for (int j = 0; j < kMergeBatch; ++j)
            ov[j] = (j < nsplit && lane < HD / 4) ? __ldcg(reinterpret_cast<const float4*>(a.o_part + (sl0 + j) * HD) + lane)
                                                  : make_float4(0.f, 0.f, 0.f, 0.f);
        const float m = warp_max_redux(m_mine);
        // an empty split, or one beyond the causal horizon, has no maximum and weighs nothing
        const float w_mine = (m_mine == -INFINITY) ? 0.f : exp2f(m_mine - m);
        const float wl_mine = w_mine * l_mine;
        float den = 0.f;
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < kMergeBatch; ++j) {
            const float w = __shfl_sync(0xffffffffu, w_mine, j);
            den += __shfl_sync(0xffffffffu, wl_mine, j);
            num.x += w * ov[j].x; num.y += w * ov[j].y; num.z += w * ov[j].z; num.w += w * ov[j].w;
        }
        for (int j = kMergeBatch; j < nsplit; ++j) {             // more splits than one batch holds: one by one
            const float w = __shfl_sync(0xffffffffu, w_mine, j);
            den += __shfl_sync(0xffffffffu, wl_mine, j);
            if (lane < HD / 4) {
                const float4 o = __ldcg(reinterpret_cast<const float4*>(a.o_part + (sl0 + j) * HD) + lane);
                num.x += w * o.x; num.y += w * o.y; num.z += w * o.z; num.w += w * o.w;
            }
        }
        if (lane < HD / 4) {
            const int rho = rho0 + rl, gq = rho / rows, r_in = rho % rows;
            const int col = (kvh * G + gq) * HD + lane * 4;
            const float inv = 1.f / den;
            if (a.xd_tbs > 0) {
                xd_store_one(a.xf_out, row0 + r_in, col, num.x * inv, KSo, a.xd_tbs);
                xd_store_one(a.xf_out, row0 + r_in, col + 1, num.y * inv, KSo, a.xd_tbs);
                xd_store_one(a.xf_out, row0 + r_in, col + 2, num.z * inv, KSo, a.xd_tbs);
                xd_store_one(a.xf_out, row0 + r_in, col + 3, num.w * inv, KSo, a.xd_tbs);
            } else {
                xf_store_pair(reinterpret_cast<uint32_t*>(a.xf_out), row0 + r_in, col, num.x * inv, num.y * inv, KSo, NTo);
                xf_store_pair(reinterpret_cast<uint32_t*>(a.xf_out), row0 + r_in, col + 2, num.z * inv, num.w * inv, KSo, NTo);
            }
        }
    }
}

}  // namespace pipesd
