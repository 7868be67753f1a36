// Multi-query decode attention over a paged bf16 KV cache: each request contributes a short chunk
// of query rows (the pending token plus its k drafts) that attend to the cached prefix and, causally,
// to each other.  The keys are cut into 8 to 10 splits ("split-K") handled by the CTAs of a thread-block
// cluster; every CTA produces an un-normalised partial output with its running max and sum in its own
// shared memory, and after a cluster barrier the partials are merged over distributed shared memory and
// written straight into the output projection's input format -- no partial results in global memory and
// no separate merge kernel (requests of 4096 keys and more use several clusters and one more merge step).
// Tiles of keys that were cached before this pass do not depend on the preceding QKV projection, so their
// copies are issued before the dependent-launch wait.
//
// One CTA (4 warps) = one KV head of one request x one split x up to 64 query rows, where the rows are
// all (query head of the group, chunk row) pairs that share the KV head (GQA).  K and V tiles of 64 keys
// travel global -> shared by bulk copies in a two-stage ring: the rows of a page that belong to one KV head
// are contiguous in the pool, so the lanes of one warp issue one copy per page and K|V and every thread waits on the
// stage's barrier (the pool stores every row with its 16-byte chunks XOR-permuted, so that ldmatrix is
// conflict-free on the verbatim copy).  QK^T and PV run on mma.sync m16n8k16 with fp32 accumulation; Q and
// the softmax probabilities are fp32 values split into bf16 hi + lo terms (two MMAs), K and V are the cache's
// bf16.  How the 4 warps share a tile depends on the number of 16-row tiles: 1 tile -> 4 key strips of 16,
// 2 tiles -> 2 x 2 strips of 32, 3-4 tiles -> one tile each over all 64 keys; warps that split the keys keep
// independent online-softmax states that are merged in shared memory.
#pragma once
#include "common.cuh"
#include "layers.cuh"

namespace pipesd {

constexpr int kAttnThreads = 128;
constexpr int kAttnTile = 64;       // keys per tile
constexpr int kAttnStages = 2;
constexpr int kAttnMaxRowTiles = 4; // 64 query rows per CTA
constexpr int kAttnPagesSmem = 512; // page ids of a CTA's key range kept in shared memory (longer ranges read the table)

// Wait for a stage barrier.  Bounded by a try count (each try suspends for a hardware-chosen time; 2^22 of them take
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

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

template <int HD>
struct AttnSmem {
    static constexpr int kRowBytes = HD * 2;
    static constexpr int kTileBytes = kAttnTile * kRowBytes;            // one K or V tile
    static constexpr int kStageBytes = 2 * kTileBytes;                  // K then V
    static constexpr int kQTileBytes = (HD / 16) * 2 * 512;             // A fragments hi+lo of one 16-row tile
    static constexpr int kRing = kAttnStages * kStageBytes;
    // ring | Q fragments (reused for the CTA's partial result, which needs 128 B more per row tile)
    static size_t bytes(int row_tiles) { return (size_t)kRing + (size_t)row_tiles * (kQTileBytes + 128); }
};

// Per-CTA constants shared by the mode-specialised bodies.
struct AttnCtx {
    const uint16_t* kbase;     // K row (slot 0) of page 0 for this layer and KV head
    const int32_t* bt;         // page ids of the request, indexed from bt_first: shared-memory copy of the CTA's range, or the table
    int bt_first;
    size_t page_stride;        // elements between consecutive pages of a layer
    size_t v_off;              // elements from a K row to the V row of the same slot
    int page_size;
    int k0, k1, base, rows, R, rho0;
};

__device__ __forceinline__ float fast_exp2(float x) {   // 2^x, relative error 2^-22; 2^-inf = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Two values -> packed bf16x2 hi and lo terms (a = hi + lo up to 2^-17 |a|).
__device__ __forceinline__ void split2_bf16(float a, float b, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    const float2 hf = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(a - hf.x, b - hf.y);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

// Issue (one warp) the copies of one 64-key tile into a ring stage: the rows of a page that belong to one KV head
// are contiguous in the pool (already chunk-permuted), so every page the tile touches is one bulk copy of K rows
// and one of V rows, counted in bytes on the stage's barrier; lane l takes the l-th page of the tile (at most nine).
// Rows at or beyond k1 are not copied.
template <int HD>
__device__ __forceinline__ void attn_issue_tile(const AttnCtx& c, uint32_t stage_addr, uint32_t bar, int j0) {
    const int lane = threadIdx.x & 31;
    const int j1 = min(j0 + kAttnTile, c.k1);
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)(j1 - j0) * (HD * 2) * 2);
    __syncwarp();
    const int pidx = j0 / c.page_size + lane;                          // this lane's page of the request
    const int js = max(j0, pidx * c.page_size), je = min(j1, (pidx + 1) * c.page_size);
    if (js < je) {
        const uint16_t* kp = c.kbase + (size_t)c.bt[pidx - c.bt_first] * c.page_stride + (size_t)(js - pidx * c.page_size) * HD;
        const uint32_t dst = stage_addr + (uint32_t)(js - j0) * (HD * 2);
        bulk_g2s(dst, kp, (uint32_t)(je - js) * (HD * 2), bar);
        bulk_g2s(dst + AttnSmem<HD>::kTileBytes, kp + c.v_off, (uint32_t)(je - js) * (HD * 2), bar);
    }
}

// On entry the copies of tiles 0 and 1 have been issued on the two stage barriers.  On exit the
// CTA's partial result for its (up to 64) rows is in shared memory: Fo[row][HD], Fm[row], Fl[row].
template <int HD, int RTW>
__device__ __forceinline__ void attn_body(const AttnCtx& c, const AttnCtx* c_issue, unsigned char* smem, uint32_t bars, int* err,
                                          float* __restrict__ Fo, float* __restrict__ Fm, float* __restrict__ Fl) {
    constexpr int KSW = 4 / RTW;               // key strips per tile
    constexpr int STRIP = kAttnTile / KSW;     // keys per warp per tile
    constexpr int NTS = STRIP / 8;             // score n-tiles per warp
    constexpr int KSTEPS = HD / 16;
    constexpr int NTO = HD / 8;                // output n-tiles
    using SM = AttnSmem<HD>;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int rtw = warp % RTW, strip = warp / RTW;
    const uint32_t ring = smem_u32(smem);
    const unsigned char* qs = smem + SM::kRing + rtw * SM::kQTileBytes;
    const int sk0 = strip * STRIP;
    const bool warp_active = c.rho0 + rtw * 16 < c.R;

    float o[NTO][4];
#pragma unroll
    for (int i = 0; i < NTO; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[i][e] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    // rows of this lane: rho = rho0 + rtw*16 + g (+8); r = rho % rows gives the causal horizon base + r
    int horizon[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const int rho = c.rho0 + rtw * 16 + g + 8 * hh;
        horizon[hh] = rho < c.R ? c.base + rho % c.rows : -1;   // keys j <= horizon are visible (padding rows: results unused)
    }

    const int ntiles = c.k1 > c.k0 ? (c.k1 - c.k0 + kAttnTile - 1) / kAttnTile : 0;

    for (int it = 0; it < ntiles; ++it) {
        const int stg = it % kAttnStages;
        if (it > 0) {
            __syncthreads();      // everyone is done with tile it-1: its stage can take tile it+1
            if (it + 1 < ntiles && warp == 0) {
                fence_proxy_async_smem();      // the stage was read with ordinary loads; the copy engine writes it next
                attn_issue_tile<HD>(*c_issue, ring + ((it + 1) % kAttnStages) * SM::kStageBytes,
                                    bars + 8 * ((it + 1) % kAttnStages), c.k0 + (it + 1) * kAttnTile);
            }
        }
        // a ragged last tile: its rows at and beyond k1 are not copied; V there must be finite (P is 0, but 0 * NaN
        // is not), so those rows are cleared, by everyone, in the part of the stage the copy does not touch
        const int n_valid = min(kAttnTile, c.k1 - (c.k0 + it * kAttnTile));
        if (n_valid < kAttnTile) {
            unsigned char* sp = smem + stg * SM::kStageBytes;
            for (int i = n_valid * (HD / 8) + threadIdx.x; i < kAttnTile * (HD / 8); i += kAttnThreads) {
                *reinterpret_cast<uint4*>(sp + (size_t)i * 16) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(sp + SM::kTileBytes + (size_t)i * 16) = make_uint4(0, 0, 0, 0);
            }
        }
        if (!attn_wait(bars + 8 * stg, (uint32_t)(it / kAttnStages) & 1u) && err) atomicExch(err, 3);   // tile `it` has landed
        if (n_valid < kAttnTile) __syncthreads();
        if (!warp_active) continue;
        const uint32_t kst = ring + stg * SM::kStageBytes;
        const uint32_t vst = kst + SM::kTileBytes;
        const int j0 = c.k0 + it * kAttnTile + sk0;    // first key of this warp's strip

        // ---- S = Q K^T over the strip
        constexpr bool kTwoChains = NTS <= 4;     // short strips: keep the hi and lo products in separate chains
        float s[NTS][4], s2[kTwoChains ? NTS : 1][4];
#pragma unroll
        for (int i = 0; i < NTS; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) { s[i][e] = 0.f; if (kTwoChains) s2[i][e] = 0.f; }
#pragma unroll
        for (int kp = 0; kp < KSTEPS / 2; ++kp) {
            const uint4 qh0 = *reinterpret_cast<const uint4*>(qs + (((2 * kp) * 2 + 0) * 32 + lane) * 16);
            const uint4 ql0 = *reinterpret_cast<const uint4*>(qs + (((2 * kp) * 2 + 1) * 32 + lane) * 16);
            const uint4 qh1 = *reinterpret_cast<const uint4*>(qs + (((2 * kp + 1) * 2 + 0) * 32 + lane) * 16);
            const uint4 ql1 = *reinterpret_cast<const uint4*>(qs + (((2 * kp + 1) * 2 + 1) * 32 + lane) * 16);
#pragma unroll
            for (int nt = 0; nt < NTS; ++nt) {
                const int row = sk0 + nt * 8 + (lane & 7);
                const int ch = kp * 4 + (lane >> 3);
                uint32_t b[4];
                ldmatrix_x4(b, kst + row * (HD * 2) + ((ch ^ (row & 7)) << 4));
                mma_bf16_16816(s[nt], qh0, b[0], b[1]);
                mma_bf16_16816(kTwoChains ? s2[nt] : s[nt], ql0, b[0], b[1]);
                mma_bf16_16816(s[nt], qh1, b[2], b[3]);
                mma_bf16_16816(kTwoChains ? s2[nt] : s[nt], ql1, b[2], b[3]);
            }
        }
        if (kTwoChains) {
#pragma unroll
            for (int nt = 0; nt < NTS; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) s[nt][e] += s2[nt][e];
        }
        // ---- mask (only strips that reach this pass's rows or the split's end), online softmax
        const bool need_mask = j0 + STRIP - 1 > c.base || j0 + STRIP > c.k1;     // warp-uniform
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < NTS; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int hh = e >> 1;
                if (need_mask) {
                    const int j = j0 + nt * 8 + 2 * t + (e & 1);
                    if (!(j < c.k1 && j <= horizon[hh])) s[nt][e] = -INFINITY;
                }
                mx[hh] = fmaxf(mx[hh], s[nt][e]);
            }
        float alpha[2], m_use[2];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
            mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
            const float m_new = fmaxf(m_run[hh], mx[hh]);
            m_use[hh] = m_new == -INFINITY ? 0.f : m_new;       // keeps (-inf) - (-inf) out of the exponent
            alpha[hh] = fast_exp2(m_run[hh] - m_use[hh]);       // 0 while nothing has been seen yet
            m_run[hh] = m_new;
            l_run[hh] *= alpha[hh];
        }
#pragma unroll
        for (int nt = 0; nt < NTS; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int hh = e >> 1;
                const float p = fast_exp2(s[nt][e] - m_use[hh]);  // masked: 2^-inf = 0
                s[nt][e] = p;
                l_run[hh] += p;      // per-lane partial; the quad is summed once at the end
            }
        if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {   // the running max rarely moves
#pragma unroll
            for (int i = 0; i < NTO; ++i) {
                o[i][0] *= alpha[0]; o[i][1] *= alpha[0];
                o[i][2] *= alpha[1]; o[i][3] *= alpha[1];
            }
        }
        // ---- O += P V over the strip's keys, P split into bf16 hi + lo
#pragma unroll
        for (int kk = 0; kk < STRIP / 16; ++kk) {
            uint4 ph, pl;
            split2_bf16(s[2 * kk][0], s[2 * kk][1], ph.x, pl.x);
            split2_bf16(s[2 * kk][2], s[2 * kk][3], ph.y, pl.y);
            split2_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1], ph.z, pl.z);
            split2_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3], ph.w, pl.w);
#pragma unroll
            for (int np = 0; np < NTO / 2; ++np) {
                const int row = sk0 + kk * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);
                const int ch = np * 2 + (lane >> 4);
                uint32_t b[4];
                ldmatrix_x4_trans(b, vst + row * (HD * 2) + ((ch ^ (row & 7)) << 4));
                mma_bf16_16816(o[2 * np], ph, b[0], b[1]);
                mma_bf16_16816(o[2 * np], pl, b[0], b[1]);
                mma_bf16_16816(o[2 * np + 1], ph, b[2], b[3]);
                mma_bf16_16816(o[2 * np + 1], pl, b[2], b[3]);
            }
        }
    }
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 1);
        l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 2);
    }

    __syncthreads();                               // every warp is done with the ring: reuse it
    // ---- leave the CTA's partial result in shared memory; merge the key strips first when the warps split the keys
    if (KSW == 1) {
        if (warp_active) {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int rl = rtw * 16 + g + 8 * hh;          // row within the CTA's row group
#pragma unroll
                for (int i = 0; i < NTO; ++i)
                    *reinterpret_cast<float2*>(Fo + (size_t)rl * HD + i * 8 + 2 * t) = make_float2(o[i][2 * hh], o[i][2 * hh + 1]);
                if (t == 0) { Fm[rl] = m_run[hh]; Fl[rl] = l_run[hh]; }
            }
        }
        return;
    }
    constexpr int MOS = HD + 8;                    // padded row: a warp's float2 stores of one n-tile fall on distinct banks
    float* mo = reinterpret_cast<float*>(smem);    // [warp][16 rows][MOS] then [warp][16] m, [warp][16] l, [warp][16] weight
    float* mm = mo + 4 * 16 * MOS;
    float* ml = mm + 4 * 16;
    float* mw = ml + 4 * 16;
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const int row = g + 8 * hh;
#pragma unroll
        for (int i = 0; i < NTO; ++i)
            *reinterpret_cast<float2*>(mo + ((size_t)warp * 16 + row) * MOS + i * 8 + 2 * t) =
                make_float2(o[i][2 * hh], o[i][2 * hh + 1]);
        if (t == 0) { mm[warp * 16 + row] = m_run[hh]; ml[warp * 16 + row] = l_run[hh]; }
    }
    __syncthreads();
    // per row: the merged maximum, every strip's weight 2^(m_strip - m) and the merged sum, once (not per column)
    if (threadIdx.x < RTW * 16) {
        const int tile = threadIdx.x / 16, row = threadIdx.x % 16;
        float m = -INFINITY;
#pragma unroll
        for (int k = 0; k < KSW; ++k) m = fmaxf(m, mm[(k * RTW + tile) * 16 + row]);
        float l = 0.f;
#pragma unroll
        for (int k = 0; k < KSW; ++k) {
            const int w = k * RTW + tile;
            const float ms = mm[w * 16 + row];
            const float wgt = (ms == -INFINITY) ? 0.f : exp2f(ms - m);
            mw[w * 16 + row] = wgt;
            l += wgt * ml[w * 16 + row];
        }
        Fm[threadIdx.x] = m;
        Fl[threadIdx.x] = l;
    }
    __syncthreads();
    // thread -> (row tile group, row, column pairs): RTW*16 rows x HD/2 pairs over 128 threads
    for (int idx = threadIdx.x; idx < RTW * 16 * (HD / 2); idx += kAttnThreads) {
        const int e = 2 * (idx % (HD / 2)), rr = idx / (HD / 2), tile = rr / 16, row = rr % 16;
        float v0 = 0.f, v1 = 0.f;
#pragma unroll
        for (int k = 0; k < KSW; ++k) {
            const int w = k * RTW + tile;
            const float wgt = mw[w * 16 + row];
            const float2 ov = *reinterpret_cast<const float2*>(mo + ((size_t)w * 16 + row) * MOS + e);
            v0 += wgt * ov.x; v1 += wgt * ov.y;
        }
        *reinterpret_cast<float2*>(Fo + (size_t)rr * HD + e) = make_float2(v0, v1);
    }
}

constexpr int kAttnSplits = 8;        // key splits per cluster of a request whose keys several clusters share
constexpr int kAttnMaxCluster = 10;   // largest cluster along x (above 8: the non-portable sizes, opted into by the host;
                                      // a B200 keeps 41 clusters of 10 of this kernel resident but only 31 of 11 or 12)

// Host: how one request's keys are split.  `resident[w - 8]` = clusters of width w (8, 9, 10) the device keeps
// resident at once for this request's shared-memory footprint (0: width unavailable); `need` = clusters the request
// launches per layer (KV heads x row groups).  One cluster of eight per 2048 keys up to four clusters; a single
// cluster widens to the smallest width that leaves each CTA the fewest 64-key tiles, as long as all the request's
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


// grid (cs * max clusters per request, n_kv_heads * row_groups, n_items), cluster (cs,1,1), 8 <= cs <= 10, block 128.
// A request uses the first it_cs <= cs CTAs of its cluster; the others hold an empty split (exact zeros in the
// merge), so a request's result does not depend on the cluster size its batch was launched with.
// A request whose keys are shared by several clusters (long contexts) takes one more step: every cluster
// writes its merged partial to global memory and the last cluster to arrive (atomic ticket, nobody waits)
// merges those.
template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 3) attn_kernel(const float* __restrict__ q, PassMeta meta,
                                                            const uint16_t* __restrict__ kv_pool, int layer,
                                                            int n_pages, int page_size, int M, int Hq, int Hkv,
                                                            int q_tiles_smem, int row_groups, float* __restrict__ o_part,
                                                            float* __restrict__ m_part, float* __restrict__ l_part,
                                                            int* __restrict__ tickets, uint16_t* __restrict__ xf_out,
                                                            int xu_layout, int* __restrict__ err, const L2Prefetch pf) {
    extern __shared__ __align__(128) unsigned char smem[];
    using SM = AttnSmem<HD>;
    pdl_launch_dependents();
    // attention leaves most of the HBM bandwidth unused: the output projection's weights come into L2 meanwhile
    if (threadIdx.x == 0)
        l2_prefetch_issue(pf, (int)((blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x),
                          (int)(gridDim.x * gridDim.y * gridDim.z));
    const int item = blockIdx.z;
    const int cs = (int)cluster_nctaid_x();
    const int cl = blockIdx.x / cs, rank = blockIdx.x % cs;        // cluster of this (request, head), rank in it
    const int ncl = meta.it_nsplit[item];                          // clusters that share this request's keys
    if (cl >= ncl) return;                                         // taken by a whole cluster or by none
    const int S = meta.it_cs[item];                                // key splits per cluster of this request (<= cs)
    const int sp = cl * S + rank;                                  // key split of this CTA (rank < S)
    const int kvh = blockIdx.y % Hkv, rg = blockIdx.y / Hkv;
    const int G = Hq / Hkv;
    AttnCtx c;
    c.rows = meta.it_rows[item];
    c.R = G * c.rows;
    c.rho0 = rg * (kAttnMaxRowTiles * 16);
    int row_tiles = (c.R - c.rho0 + 15) / 16;
    row_tiles = row_tiles > kAttnMaxRowTiles ? kAttnMaxRowTiles : row_tiles;
    // the whole cluster shares (item, head, row group): these exits are taken by all CTAs of the cluster or by none
    if (c.rho0 >= c.R || row_tiles > q_tiles_smem) return;
    c.base = meta.it_base[item];
    const int total = c.base + c.rows, chunk = meta.it_chunk[item];
    c.k0 = rank < S ? min(sp * chunk, total) : total;
    c.k1 = min(c.k0 + chunk, total);
    c.kbase = kv_pool + kv_index(layer, n_pages, 0, 0, Hkv, kvh, page_size, 0, HD, 0);
    c.page_stride = (size_t)2 * Hkv * page_size * HD;
    c.v_off = (size_t)Hkv * page_size * HD;
    c.page_size = page_size;
    c.bt = meta.block_tab + (size_t)meta.it_slot[item] * meta.max_pages;
    c.bt_first = 0;
    // The page ids of this CTA's key range go to shared memory once: a tile's copies then start without a trip to
    // the block table first (that lookup, ahead of every tile's loads, cost about a microsecond per tile).
    __shared__ int s_pages[kAttnPagesSmem];
    if (c.k1 > c.k0) {
        const int p_first = c.k0 / page_size, n_pg = (c.k1 - 1) / page_size - p_first + 1;
        if (n_pg <= kAttnPagesSmem) {                              // uniform over the CTA
            for (int i = threadIdx.x; i < n_pg; i += kAttnThreads) s_pages[i] = c.bt[p_first + i];
            __syncthreads();
            c.bt = s_pages;
            c.bt_first = p_first;
        }
    }
    const int row0 = meta.it_row0[item];
    const uint32_t ring = smem_u32(smem);

    // Tiles made only of keys cached before this pass do not depend on the QKV projection that precedes this
    // kernel: their copies are issued now, the others after the dependency has resolved.
    __shared__ AttnCtx s_ctx;      // warp 0's copy: what issuing a tile needs stays out of everyone's registers
    __shared__ __align__(8) unsigned long long s_bars[kAttnStages];
    const uint32_t bars = smem_u32(s_bars);
    const int ntiles = c.k1 > c.k0 ? (c.k1 - c.k0 + kAttnTile - 1) / kAttnTile : 0;
    const bool early0 = ntiles > 0 && min(c.k0 + kAttnTile, c.k1) <= c.base;
    const bool early1 = ntiles > 1 && min(c.k0 + 2 * kAttnTile, c.k1) <= c.base;
    if (threadIdx.x < 32) {          // warp 0 issues every tile
        if (threadIdx.x == 0) {
            s_ctx = c;
            for (int i = 0; i < kAttnStages; ++i) mbar_init(bars + 8 * i, 1);
            fence_mbar_init();
        }
        __syncwarp();
        if (early0) attn_issue_tile<HD>(s_ctx, ring, bars, c.k0);
        if (early1) attn_issue_tile<HD>(s_ctx, ring + SM::kStageBytes, bars + 8, c.k0 + kAttnTile);
    }
    pdl_wait();
    if (threadIdx.x < 32) {
        if (!early0 && ntiles > 0) attn_issue_tile<HD>(s_ctx, ring, bars, c.k0);
        if (!early1 && ntiles > 1) attn_issue_tile<HD>(s_ctx, ring + SM::kStageBytes, bars + 8, c.k0 + kAttnTile);
    }

    // ---- stage Q (scaled by 1/sqrt(hd)) as split-bf16 A fragments: [tile][k16 step][hi|lo][lane] uint4
    const float scale = rsqrtf((float)HD) * 1.4426950408889634f;   // scores in the log2 domain: p = 2^(s - m)
    uint4* qsm = reinterpret_cast<uint4*>(smem + SM::kRing);
#pragma unroll 2
    for (int idx = threadIdx.x; idx < row_tiles * (HD / 16) * 32; idx += kAttnThreads) {
        const int lane = idx & 31, ks = (idx >> 5) % (HD / 16), tile = idx / (32 * (HD / 16));
        const int g = lane >> 2, t = lane & 3;
        float v[8];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int rho = c.rho0 + tile * 16 + g + 8 * hh;
            float2 a = make_float2(0.f, 0.f), b = make_float2(0.f, 0.f);
            if (rho < c.R) {
                const int gq = rho / c.rows, r = rho % c.rows;
                const float* qp = q + ((size_t)(row0 + r) * Hq + kvh * G + gq) * HD + ks * 16 + 2 * t;
                a = *reinterpret_cast<const float2*>(qp);
                b = *reinterpret_cast<const float2*>(qp + 8);
            }
            v[2 * hh] = a.x * scale; v[2 * hh + 1] = a.y * scale;
            v[4 + 2 * hh] = b.x * scale; v[4 + 2 * hh + 1] = b.y * scale;
        }
        uint16_t h[8], l[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) split_bf16(v[i], h[i], l[i]);
        // A fragment order: (row g, k 2t..), (row g+8, k 2t..), (row g, k 2t+8..), (row g+8, k 2t+8..)
        qsm[((tile * (HD / 16) + ks) * 2 + 0) * 32 + lane] =
            make_uint4(pack2(h[0], h[1]), pack2(h[2], h[3]), pack2(h[4], h[5]), pack2(h[6], h[7]));
        qsm[((tile * (HD / 16) + ks) * 2 + 1) * 32 + lane] =
            make_uint4(pack2(l[0], l[1]), pack2(l[2], l[3]), pack2(l[4], l[5]), pack2(l[6], l[7]));
    }
    __syncthreads();

    // partial result of this CTA: takes over the Q-fragment region once the tile loop is done
    float* Fo = reinterpret_cast<float*>(smem + SM::kRing);     // [row_tiles*16][HD]
    float* Fm = Fo + row_tiles * 16 * HD;                        // [row_tiles*16]
    float* Fl = Fm + row_tiles * 16;                             // [row_tiles*16]
    if (ntiles == 0) {   // empty split: contributes nothing (finite zeros, so the merge can read it unconditionally)
        for (int i = threadIdx.x; i < row_tiles * 16; i += kAttnThreads) { Fm[i] = -INFINITY; Fl[i] = 0.f; }
        for (int i = threadIdx.x; i < row_tiles * 16 * HD; i += kAttnThreads) Fo[i] = 0.f;
    } else if (row_tiles == 1) attn_body<HD, 1>(c, &s_ctx, smem, bars, err, Fo, Fm, Fl);
    else if (row_tiles == 2) attn_body<HD, 2>(c, &s_ctx, smem, bars, err, Fo, Fm, Fl);
    else attn_body<HD, 4>(c, &s_ctx, smem, bars, err, Fo, Fm, Fl);

    // ---- merge the cluster's splits over distributed shared memory; rank r owns rows r, r+cs, ... of the group
    cluster_sync_all();
    constexpr int EPT = HD / kAttnThreads > 0 ? HD / kAttnThreads : 1;   // output columns per thread
    const uint32_t fo_a = smem_u32(Fo), fm_a = smem_u32(Fm), fl_a = smem_u32(Fl);
    const int n_rows = min(row_tiles * 16, c.R - c.rho0);
    const int KSo = (Hq * HD) / 16, NTo = xf_nt(M);
    const size_t slot0 = (size_t)meta.it_part0[item] + ((size_t)kvh * c.R + c.rho0) * ncl;   // + rl*ncl + cluster
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
                const int e = threadIdx.x + k * kAttnThreads;
                ov[k][r] = e < HD ? dsmem_ld_f32(dsmem_addr(fo_a + (uint32_t)(rl * HD + e) * 4, (uint32_t)r)) : 0.f;
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
        const int rho = c.rho0 + rl, gq = rho / c.rows, r_in = rho % c.rows;
#pragma unroll
        for (int k = 0; k < EPT; ++k) {
            const int e = threadIdx.x + k * kAttnThreads;
            if (e < HD) {
                float num = 0.f;
#pragma unroll
                for (int r = 0; r < kAttnMaxCluster; ++r) num += w[r] * ov[k][r];
                if (ncl == 1) {
                    if (xu_layout) xu_store_one(xf_out, row0 + r_in, (kvh * G + gq) * HD + e, num / den, NTo);
                    else xf_store_one(xf_out, row0 + r_in, (kvh * G + gq) * HD + e, num / den, KSo, NTo);
                }
                else o_part[(slot0 + (size_t)rl * ncl + cl) * HD + e] = num;     // un-normalised, with (m, den)
            }
        }
        if (ncl > 1 && threadIdx.x == 0) {
            m_part[slot0 + (size_t)rl * ncl + cl] = m;
            l_part[slot0 + (size_t)rl * ncl + cl] = den;
        }
    }
    __shared__ int s_last;
    if (ncl > 1) __threadfence();
    cluster_sync_all();   // nobody leaves while its shared memory may still be read; partials are published
    if (ncl == 1) return;
    // ---- several clusters share the keys: the last one to arrive merges their partials
    if (rank == 0 && threadIdx.x == 0) {
        int* ticket = tickets + ((size_t)item * Hkv + kvh) * row_groups + rg;
        const int t = atomicAdd(ticket, 1);
        const int last = (t == ncl - 1);
        if (last) *ticket = 0;                                   // self-cleaning: ready for the next launch
        const uint32_t fa = smem_u32(&s_last);
        for (int r = 0; r < cs; ++r) dsmem_st_f32(dsmem_addr(fa, (uint32_t)r), __int_as_float(last));
    }
    cluster_sync_all();
    if (!s_last) return;
    __threadfence();
    for (int rl = rank; rl < n_rows; rl += cs) {
        float ms[kMaxSplits / kAttnSplits], ls[kMaxSplits / kAttnSplits], ov[EPT][kMaxSplits / kAttnSplits];
#pragma unroll
        for (int j = 0; j < kMaxSplits / kAttnSplits; ++j) {
            const bool on = j < ncl;
            const size_t sl = slot0 + (size_t)rl * ncl + j;
            ms[j] = on ? __ldcg(m_part + sl) : -INFINITY;
            ls[j] = on ? __ldcg(l_part + sl) : 0.f;
#pragma unroll
            for (int k = 0; k < EPT; ++k) {
                const int e = threadIdx.x + k * kAttnThreads;
                ov[k][j] = (on && e < HD) ? __ldcg(o_part + sl * HD + e) : 0.f;
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
        const int rho = c.rho0 + rl, gq = rho / c.rows, r_in = rho % c.rows;
#pragma unroll
        for (int k = 0; k < EPT; ++k) {
            const int e = threadIdx.x + k * kAttnThreads;
            if (e < HD) {
                float num = 0.f;
#pragma unroll
                for (int j = 0; j < kMaxSplits / kAttnSplits; ++j) num += w[j] * ov[k][j];
                if (xu_layout) xu_store_one(xf_out, row0 + r_in, (kvh * G + gq) * HD + e, num / den, NTo);
                else xf_store_one(xf_out, row0 + r_in, (kvh * G + gq) * HD + e, num / den, KSo, NTo);
            }
        }
    }
}

static inline size_t attn_smem_bytes(int hd, int row_tiles) {
    return hd == 128 ? AttnSmem<128>::bytes(row_tiles) : AttnSmem<64>::bytes(row_tiles);
}

}  // namespace pipesd
