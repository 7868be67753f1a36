// Element-wise / per-row kernels of the verify pass: embedding gather, split-K reduction fused with
// the residual add and RMSNorm, rotary embedding fused with the KV-page append, SwiGLU gate.
#pragma once
#include "common.cuh"

namespace pipesd {

// Per-pass metadata that lives in device memory (uploaded once per call).
struct PassMeta {
    const int32_t* row_item;   // [M] batch item of each row
    const int32_t* row_pos;    // [M] absolute position of each row in its request
    const int32_t* row_tok;    // [M] token id of each row
    const int32_t* it_slot;    // [n_items] request slot (row of the block table)
    const int32_t* it_row0;    // [n_items] first row of the item
    const int32_t* it_rows;    // [n_items] rows of the item (k+1)
    const int32_t* it_base;    // [n_items] cached positions before this pass
    const int32_t* it_nsplit;  // [n_items] KV splits
    const int32_t* it_chunk;   // [n_items] keys per split (multiple of the page size)
    const int32_t* it_part0;   // [n_items] first slot of the item in the attention partial arrays
    const int32_t* block_tab;  // [max_requests][max_pages] page ids, indexed by request slot
    int max_pages;
};

// x_new = (first layer ? bf16 embedding row : x) + sum_s part[s]   (residual stream, fp32)
// h     = x_new * rsqrt(mean(x_new^2) + eps) * gain
// One CTA per row.  The sum over split-K partials is taken in slice order (deterministic).
__global__ void __launch_bounds__(256) add_norm_kernel(float* __restrict__ x, const uint16_t* __restrict__ emb,
                                                       const int32_t* __restrict__ row_tok,
                                                       const float* __restrict__ part, int S, int M,
                                                       const float* __restrict__ gain, float eps, int d,
                                                       float* __restrict__ h) {
    const int row = blockIdx.x;
    __shared__ float red[8];
    float ss = 0.f;
    float* xr = x + (size_t)row * d;
    for (int e = threadIdx.x; e < d; e += 256) {
        float v = emb ? bf16_bits_to_f32(emb[(size_t)row_tok[row] * d + e]) : xr[e];
        for (int s = 0; s < S; ++s) v += part[((size_t)s * M + row) * d + e];
        xr[e] = v;
        ss += v * v;
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const float r = rsqrtf(tot / (float)d + eps);
    for (int e = threadIdx.x; e < d; e += 256) h[(size_t)row * d + e] = xr[e] * r * gain[e];
}

// cos/sin of pos * base^(-2j/hd), evaluated in fp64 (positions reach 10^4, fp32 angles would lose
// three digits), stored fp32 [M][hd/2].
__global__ void rope_table_kernel(const int32_t* __restrict__ row_pos, int M, int hd, double log_base,
                                  float* __restrict__ cs, float* __restrict__ sn) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    int half = hd / 2;
    if (i >= M * half) return;
    int row = i / half, j = i % half;
    double theta = exp(-2.0 * (double)j / (double)hd * log_base);
    double ang = (double)row_pos[row] * theta;
    double s, c;
    sincos(ang, &s, &c);
    cs[i] = (float)c;
    sn[i] = (float)s;
}

// Sum the QKV split-K partials, rotate q and k ("rotate-half": element j pairs with j + hd/2),
// keep q in fp32, round k and v to bf16 and write them into the request's KV pages.
// grid (M, n_q_heads + 2*n_kv_heads), block hd/2.
__global__ void rope_kv_kernel(const float* __restrict__ part, int S, int M, int Hq, int Hkv, int hd,
                               const float* __restrict__ cs, const float* __restrict__ sn, PassMeta meta,
                               float* __restrict__ qout, uint16_t* __restrict__ kv_pool, int layer,
                               int n_pages, int page_size) {
    const int row = blockIdx.x, head = blockIdx.y, j = threadIdx.x, half = hd / 2;
    const int Nqkv = (Hq + 2 * Hkv) * hd;
    const int col = head * hd + j;
    float a = 0.f, b = 0.f;
    for (int s = 0; s < S; ++s) {
        const float* p = part + ((size_t)s * M + row) * Nqkv + col;
        a += p[0];
        b += p[half];
    }
    if (head < Hq + Hkv) {  // q and k heads are rotated
        float c = cs[row * half + j], sgn = sn[row * half + j];
        float ra = a * c - b * sgn, rb = b * c + a * sgn;
        a = ra;
        b = rb;
    }
    if (head < Hq) {
        float* q = qout + (size_t)row * Hq * hd + head * hd;
        q[j] = a;
        q[j + half] = b;
        return;
    }
    const int item = meta.row_item[row], pos = meta.row_pos[row];
    const int page = meta.block_tab[(size_t)meta.it_slot[item] * meta.max_pages + pos / page_size];
    const int kv = head < Hq + Hkv ? 0 : 1;
    const int kvh = kv ? head - Hq - Hkv : head - Hq;
    uint16_t* dst = kv_pool + kv_index(layer, n_pages, page, kv, Hkv, kvh, page_size, pos % page_size, hd, 0);
    dst[j] = f32_to_bf16_bits(a);
    dst[j + half] = f32_to_bf16_bits(b);
}

// act = silu(sum_s gate_s) * sum_s up_s ; partials are [S][M][2F] with gate in [0,F), up in [F,2F).
__global__ void silu_mul_kernel(const float* __restrict__ part, int S, int M, int F, float* __restrict__ act) {
    size_t n = (size_t)M * F;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        size_t row = i / F, f = i % F;
        float g = 0.f, u = 0.f;
        for (int s = 0; s < S; ++s) {
            const float* p = part + ((size_t)s * M + row) * 2 * F;
            g += p[f];
            u += p[F + f];
        }
        act[i] = g / (1.f + expf(-g)) * u;
    }
}

}  // namespace pipesd
