// Per-row helper kernels of the verify pass: embedding gather (start of the residual stream) and the
// rotary-embedding angle table.  Everything else element-wise is fused into the GEMM epilogues.
#pragma once
#include "common.cuh"
#include "gemm.cuh"

namespace pipesd {

// x = bf16 embedding row (residual stream, fp32); xf = x * gain of the first RMSNorm as split-bf16
// fragments (or, with tbs > 0, as an xd array of that token block size); ssq[0][row] = sum x^2, ssq[b > 0][row] = 0
// (the consumer adds n_ssq block sums up).
// One CTA of 1024 threads per row, four columns per thread.
constexpr int kEmbedThreads = 1024;
constexpr int kEmbedMaxVec = 2;   // float4 per thread: d <= 8192
__global__ void __launch_bounds__(kEmbedThreads) embed_kernel(float* __restrict__ x, const uint16_t* __restrict__ emb,
                                                              const int32_t* __restrict__ row_tok, int M,
                                                              const float* __restrict__ gain, int d,
                                                              uint32_t* __restrict__ xf_out, float* __restrict__ ssq,
                                                              int n_ssq, int tbs) {
    pdl_wait();
    pdl_launch_dependents();
    const int row = blockIdx.x;
    __shared__ float red[kEmbedThreads / 32];
    float ss = 0.f;
    float* xr = x + (size_t)row * d;
    const int KS = d / 16, NT = xf_nt(M);
#pragma unroll
    for (int i = 0; i < kEmbedMaxVec; ++i) {
        const int e = (threadIdx.x + i * kEmbedThreads) * 4;
        if (e < d) {
            const uint2 b = *reinterpret_cast<const uint2*>(emb + (size_t)row_tok[row] * d + e);
            const float4 a = make_float4(__uint_as_float(b.x << 16), __uint_as_float(b.x & 0xffff0000u),
                                         __uint_as_float(b.y << 16), __uint_as_float(b.y & 0xffff0000u));
            *reinterpret_cast<float4*>(xr + e) = a;
            ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
            const float4 g = *reinterpret_cast<const float4*>(gain + e);
            if (tbs > 0) {
                uint16_t* xd = reinterpret_cast<uint16_t*>(xf_out);
                xd_store_one(xd, row, e, a.x * g.x, KS, tbs);
                xd_store_one(xd, row, e + 1, a.y * g.y, KS, tbs);
                xd_store_one(xd, row, e + 2, a.z * g.z, KS, tbs);
                xd_store_one(xd, row, e + 3, a.w * g.w, KS, tbs);
            } else {
                xf_store_pair(xf_out, row, e, a.x * g.x, a.y * g.y, KS, NT);
                xf_store_pair(xf_out, row, e + 2, a.z * g.z, a.w * g.w, KS, NT);
            }
        }
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < n_ssq) {
        float tot = 0.f;
        if (threadIdx.x == 0) {
#pragma unroll
            for (int w = 0; w < kEmbedThreads / 32; ++w) tot += red[w];
        }
        ssq[(size_t)threadIdx.x * M + row] = tot;
    }
}

// cos/sin of pos * base^(-2j/hd), evaluated in fp64 (positions reach 10^4, fp32 angles would lose
// three digits), stored fp32 [M][hd/2]; and, per row, the element offset of its K row (head 0) inside a
// layer of the paged pool, so that the QKV epilogue appends K/V without walking the page table.
__global__ void rope_table_kernel(PassMeta meta, int M, int hd, double log_base, float* __restrict__ cs,
                                  float* __restrict__ sn, long long* __restrict__ row_kvoff, int n_pages, int Hkv,
                                  int page_size) {
    pdl_wait();
    pdl_launch_dependents();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    int half = hd / 2;
    if (i >= M * half) return;
    int row = i / half, j = i % half;
    const int pos = meta.row_pos[row];
    if (j == 0) {
        const int item = meta.row_item[row];
        const int page = meta.block_tab[(size_t)meta.it_slot[item] * meta.max_pages + pos / page_size];
        row_kvoff[row] = (long long)kv_index(0, n_pages, page, 0, Hkv, 0, page_size, pos % page_size, hd, 0);
    }
    double theta = exp(-2.0 * (double)j / (double)hd * log_base);
    double ang = (double)pos * theta;
    double s, c;
    sincos(ang, &s, &c);
    cs[i] = (float)c;
    sn[i] = (float)s;
}

// Self-test of the bounded-wait convention every kernel of the library follows: poll a flag that nothing ever sets,
// give up when the time limit is reached, record that in the device error word and return normally.  The host then
// reports the error at its next synchronisation and the context stays usable.
__global__ void wait_never_kernel(const int* __restrict__ flag, int* __restrict__ err, unsigned long long limit_ns) {
    if (threadIdx.x != 0) return;
    const unsigned long long t0 = global_ns();
    bool seen = false;
    for (unsigned it = 0; !seen; ++it) {
        seen = *reinterpret_cast<const volatile int*>(flag) != 0;
        if (!seen && global_ns() - t0 > limit_ns) break;
        if (it > (1u << 28)) break;       // an iteration cap on top of the clock
    }
    if (!seen) atomicExch(err, 77);
}

}  // namespace pipesd
