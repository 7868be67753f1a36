// Multi-query decode attention over a paged bf16 KV cache: each request contributes a short chunk
// of query rows (the pending token plus its k drafts) that attend to the cached prefix and, causally,
// to each other.  The prefix is cut into splits ("split-K"); every split produces an un-normalised
// partial output with its running max and sum, and a second kernel merges the splits.
#pragma once
#include "common.cuh"
#include "layers.cuh"

namespace pipesd {

constexpr int kAttnThreads = 128;
constexpr int kAttnTile = 128;  // keys per inner tile

// grid (max_nsplit, n_q_heads, n_items), block 128.  One CTA: one query head of one request against
// one split of its keys.  Thread t scores key t of the tile against all rows, a warp per row does the
// online-softmax update, then thread (e, row group) accumulates P.V for output dimension e.
template <int HD>
__global__ void __launch_bounds__(kAttnThreads) attn_split_kernel(const float* __restrict__ q, PassMeta meta,
                                                                  const uint16_t* __restrict__ kv_pool,
                                                                  int layer, int n_pages, int page_size, int Hq,
                                                                  int Hkv, float* __restrict__ o_part,
                                                                  float* __restrict__ m_part,
                                                                  float* __restrict__ l_part) {
    pdl_wait();
    pdl_launch_dependents();
    constexpr int RG = kAttnThreads / HD;          // row groups in the P.V phase
    constexpr int RPT = kMaxItemRows / RG;         // rows per thread in the P.V phase
    const int item = blockIdx.z, h = blockIdx.y, sp = blockIdx.x;
    const int nsplit = meta.it_nsplit[item];
    if (sp >= nsplit) return;
    const int rows = meta.it_rows[item], row0 = meta.it_row0[item], base = meta.it_base[item];
    const int total = base + rows, chunk = meta.it_chunk[item];
    const int k0 = sp * chunk, k1 = min(k0 + chunk, total);
    const int kvh = h / (Hq / Hkv);
    const int32_t* bt = meta.block_tab + (size_t)meta.it_slot[item] * meta.max_pages;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    extern __shared__ float sm[];
    float* Qs = sm;                                   // [32][HD]
    float* Ss = Qs + kMaxItemRows * HD;               // [32][kAttnTile]
    float* m_s = Ss + kMaxItemRows * kAttnTile;       // [32]
    float* l_s = m_s + kMaxItemRows;
    float* al_s = l_s + kMaxItemRows;
    size_t* voff = reinterpret_cast<size_t*>(al_s + kMaxItemRows);  // [kAttnTile]

    const float scale = rsqrtf((float)HD);
    for (int i = tid; i < rows * HD; i += kAttnThreads) {
        int r = i / HD, e = i % HD;
        Qs[i] = q[((size_t)(row0 + r) * Hq + h) * HD + e] * scale;
    }
    if (tid < kMaxItemRows) { m_s[tid] = -INFINITY; l_s[tid] = 0.f; }
    float o[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) o[i] = 0.f;
    const int e_out = tid % HD, rg = tid / HD;
    __syncthreads();

    for (int j0 = k0; j0 < k1; j0 += kAttnTile) {
        const int nkeys = min(kAttnTile, k1 - j0);
        // phase 1: scores of key (j0 + tid) against every row
        if (tid < nkeys) {
            const int j = j0 + tid;
            const int page = bt[j / page_size], slot = j % page_size;
            const size_t koff = kv_index(layer, n_pages, page, 0, Hkv, kvh, page_size, slot, HD, 0);
            voff[tid] = kv_index(layer, n_pages, page, 1, Hkv, kvh, page_size, slot, HD, 0);
            uint4 kr[HD / 8];
            const uint4* kp = reinterpret_cast<const uint4*>(kv_pool + koff);
#pragma unroll
            for (int i = 0; i < HD / 8; ++i) kr[i] = kp[i];
            for (int r = 0; r < rows; ++r) {
                const float4* qr = reinterpret_cast<const float4*>(Qs + r * HD);
                float acc = 0.f;
#pragma unroll
                for (int i = 0; i < HD / 8; ++i) {
                    float4 qa = qr[2 * i], qb = qr[2 * i + 1];
                    uint4 kk = kr[i];
                    acc += qa.x * __uint_as_float(kk.x << 16) + qa.y * __uint_as_float(kk.x & 0xffff0000u);
                    acc += qa.z * __uint_as_float(kk.y << 16) + qa.w * __uint_as_float(kk.y & 0xffff0000u);
                    acc += qb.x * __uint_as_float(kk.z << 16) + qb.y * __uint_as_float(kk.z & 0xffff0000u);
                    acc += qb.z * __uint_as_float(kk.w << 16) + qb.w * __uint_as_float(kk.w & 0xffff0000u);
                }
                Ss[r * kAttnTile + tid] = (j <= base + r) ? acc : -INFINITY;   // causal inside the chunk
            }
        } else {
            for (int r = 0; r < rows; ++r) Ss[r * kAttnTile + tid] = -INFINITY;
        }
        __syncthreads();
        // phase 2: online softmax, one warp per row
        for (int r = warp; r < rows; r += kAttnThreads / 32) {
            float v[kAttnTile / 32];
            float mx = -INFINITY;
#pragma unroll
            for (int i = 0; i < kAttnTile / 32; ++i) { v[i] = Ss[r * kAttnTile + lane + 32 * i]; mx = fmaxf(mx, v[i]); }
            mx = warp_max(mx);
            const float m_old = m_s[r], m_new = fmaxf(m_old, mx);
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < kAttnTile / 32; ++i) {
                float p = (m_new == -INFINITY) ? 0.f : expf(v[i] - m_new);
                Ss[r * kAttnTile + lane + 32 * i] = p;
                sum += p;
            }
            sum = warp_sum(sum);
            if (lane == 0) {
                float al = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
                al_s[r] = al;
                l_s[r] = l_s[r] * al + sum;
                m_s[r] = m_new;
            }
        }
        __syncthreads();
        // phase 3: o[r][e] = o[r][e]*alpha[r] + sum_t P[r][t] V[t][e]
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            int r = i * RG + rg;
            if (r < rows) o[i] *= al_s[r];
        }
        for (int tk = 0; tk < nkeys; ++tk) {
            const float v = bf16_bits_to_f32(kv_pool[voff[tk] + e_out]);
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                int r = i * RG + rg;
                if (r < rows) o[i] += Ss[r * kAttnTile + tk] * v;
            }
        }
        __syncthreads();
    }
    const int part0 = meta.it_part0[item];
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        int r = i * RG + rg;
        if (r < rows) {
            size_t slot = (size_t)part0 + ((size_t)r * Hq + h) * nsplit + sp;
            o_part[slot * HD + e_out] = o[i];
            if (e_out == 0) { m_part[slot] = m_s[r]; l_part[slot] = l_s[r]; }
        }
    }
}

static inline size_t attn_smem_bytes(int hd) {
    return sizeof(float) * (kMaxItemRows * hd + kMaxItemRows * kAttnTile + 3 * kMaxItemRows) +
           sizeof(size_t) * kAttnTile;
}

// Merge the splits: out = sum_s e^{m_s - m} o_s / sum_s e^{m_s - m} l_s, stored as split-bf16 B fragments
// for the output projection (column index = head * hd + e).  grid (M, n_q_heads), block hd.
__global__ void attn_combine_kernel(const float* __restrict__ o_part, const float* __restrict__ m_part,
                                    const float* __restrict__ l_part, PassMeta meta, int M, int Hq, int hd,
                                    uint32_t* __restrict__ xf_out) {
    pdl_wait();
    pdl_launch_dependents();
    const int row = blockIdx.x, h = blockIdx.y, e = threadIdx.x;
    const int item = meta.row_item[row];
    const int r = row - meta.it_row0[item], nsplit = meta.it_nsplit[item];
    const size_t slot0 = (size_t)meta.it_part0[item] + ((size_t)r * Hq + h) * nsplit;
    float m = -INFINITY;
    for (int s = 0; s < nsplit; ++s) m = fmaxf(m, m_part[slot0 + s]);
    float num = 0.f, den = 0.f;
#pragma unroll 4
    for (int s = 0; s < nsplit; ++s) {
        const float ms = m_part[slot0 + s];
        const float w = (ms == -INFINITY) ? 0.f : expf(ms - m);   // a split wholly beyond the causal horizon
        num += w * o_part[(slot0 + s) * hd + e];
        den += w * l_part[slot0 + s];
    }
    const float v = num / den;
    const float v1 = __shfl_down_sync(0xffffffffu, v, 1);
    if ((e & 1) == 0) xf_store_pair(xf_out, row, h * hd + e, v, v1, (Hq * hd) / 16, xf_nt(M));
}

}  // namespace pipesd
