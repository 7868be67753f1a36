// Element-wise / per-row kernels of the verify pass: embedding gather, split-K reduction fused with
// the residual add and RMSNorm, rotary embedding fused with the KV-page append, SwiGLU gate.
#pragma once
#include "common.cuh"
#include "gemm.cuh"

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

// x_new = (first layer ? bf16 embedding row : x) + sum_s part[s]   (residual stream, fp32, written back)
// h     = x_new * rsqrt(mean(x_new^2) + eps) * gain                 (written as split-bf16 B fragments)
// One CTA of 1024 threads per row, four columns per thread.  The sum over split-K partials is taken in
// slice order (deterministic); the loads of all slices are independent, so they overlap.
constexpr int kNormThreads = 1024;
constexpr int kNormMaxVec = 2;   // float4 per thread: d <= 8192
__global__ void __launch_bounds__(kNormThreads) add_norm_kernel(float* __restrict__ x, const uint16_t* __restrict__ emb,
                                                                const int32_t* __restrict__ row_tok,
                                                                const float* __restrict__ part, int S, int M,
                                                                const float* __restrict__ gain, float eps, int d,
                                                                uint32_t* __restrict__ xf_out) {
    pdl_wait();
    pdl_launch_dependents();
    const int row = blockIdx.x;
    __shared__ float red[kNormThreads / 32];
    float4 v[kNormMaxVec];
    float ss = 0.f;
    float* xr = x + (size_t)row * d;
#pragma unroll
    for (int i = 0; i < kNormMaxVec; ++i) {
        const int e = (threadIdx.x + i * kNormThreads) * 4;
        if (e < d) {
            float4 a;
            if (emb) {
                const uint2 b = *reinterpret_cast<const uint2*>(emb + (size_t)row_tok[row] * d + e);
                a = make_float4(__uint_as_float(b.x << 16), __uint_as_float(b.x & 0xffff0000u),
                                __uint_as_float(b.y << 16), __uint_as_float(b.y & 0xffff0000u));
            } else {
                a = *reinterpret_cast<const float4*>(xr + e);
            }
#pragma unroll 4
            for (int s = 0; s < S; ++s) {
                const float4 p = *reinterpret_cast<const float4*>(part + ((size_t)s * M + row) * d + e);
                a.x += p.x; a.y += p.y; a.z += p.z; a.w += p.w;
            }
            *reinterpret_cast<float4*>(xr + e) = a;
            ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
            v[i] = a;
        }
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kNormThreads / 32; ++w) tot += red[w];
    const float r = rsqrtf(tot / (float)d + eps);
    const int KS = d / 16, NT = xf_nt(M);
#pragma unroll
    for (int i = 0; i < kNormMaxVec; ++i) {
        const int e = (threadIdx.x + i * kNormThreads) * 4;
        if (e < d) {
            const float4 g = *reinterpret_cast<const float4*>(gain + e);
            xf_store_pair(xf_out, row, e, v[i].x * r * g.x, v[i].y * r * g.y, KS, NT);
            xf_store_pair(xf_out, row, e + 2, v[i].z * r * g.z, v[i].w * r * g.w, KS, NT);
        }
    }
}

// cos/sin of pos * base^(-2j/hd), evaluated in fp64 (positions reach 10^4, fp32 angles would lose
// three digits), stored fp32 [M][hd/2].
__global__ void rope_table_kernel(const int32_t* __restrict__ row_pos, int M, int hd, double log_base,
                                  float* __restrict__ cs, float* __restrict__ sn) {
    pdl_wait();
    pdl_launch_dependents();
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
    pdl_wait();
    pdl_launch_dependents();
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

// act = silu(sum_s gate_s) * sum_s up_s, stored as split-bf16 B fragments for the down projection.
// Partials are [S][M][2F] with gate in [0,F), up in [F,2F).  One thread per (row, even column).
__global__ void silu_mul_kernel(const float* __restrict__ part, int S, int M, int F, uint32_t* __restrict__ xf_out) {
    pdl_wait();
    pdl_launch_dependents();
    const size_t n = (size_t)M * (F / 2);
    const int KS = F / 16, NT = xf_nt(M);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int row = (int)(i / (F / 2)), f = 2 * (int)(i % (F / 2));
        float2 g = make_float2(0.f, 0.f), u = make_float2(0.f, 0.f);
#pragma unroll 4
        for (int s = 0; s < S; ++s) {
            const float* p = part + ((size_t)s * M + row) * 2 * F + f;
            const float2 a = *reinterpret_cast<const float2*>(p), b = *reinterpret_cast<const float2*>(p + F);
            g.x += a.x; g.y += a.y; u.x += b.x; u.y += b.y;
        }
        xf_store_pair(xf_out, row, f, g.x / (1.f + expf(-g.x)) * u.x, g.y / (1.f + expf(-g.y)) * u.y, KS, NT);
    }
}

}  // namespace pipesd
