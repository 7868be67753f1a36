// Small-M weight-streaming GEMM: y[M,N] = x[M,K] . W[N,K]^T, bf16 W (read once from HBM), fp32 x.
//
// The weight matrix is the wide operand: a 16-row x 16-column tile of W is the A fragment of a
// warp-level m16n8k16 MMA and the (few) token rows are the narrow N dimension.  W is repacked once
// at context creation into fragment order, so that a warp's 32 lanes read one contiguous 512-byte
// block per tile with 16-byte loads straight into the registers the MMA consumes -- no shared
// memory on the weight path.  Each lane keeps kDepth such loads in flight.
// Activations stay fp32 outside; inside they are split into bf16 hi + lo terms (two MMAs into the
// same fp32 accumulator), staged once per CTA in shared memory in B-fragment order.
// Work split: CTA = (128-row block of W, K slice, 32-token block); partial sums of the K slices go
// to a scratch array [S][M][N] that the consuming kernel adds up in fixed order (deterministic).
#pragma once
#include "common.cuh"

namespace pipesd {

constexpr int kGemmThreads = 256;  // 8 warps = 8 row tiles of 16 = 128 rows of W per CTA
constexpr int kGemmDepth = 8;      // 16-byte weight loads in flight per lane
constexpr int kGemmSmemCap = 100 * 1024;

struct GemmPlan {
    int NT;      // n8 token tiles per token block (1..4)
    int TB;      // token blocks
    int RB;      // 128-row blocks
    int S;       // K slices
    int KS;      // k16 steps in K
    size_t smem; // dynamic shared memory per CTA
};

// Host: choose the K split so that the grid fills whole waves of kWaveCtas CTAs.
static inline GemmPlan gemm_plan(int M, int N, int K) {
    GemmPlan p;
    int nt = (M + 7) / 8;
    p.NT = nt > 4 ? 4 : (nt < 1 ? 1 : nt);
    p.TB = (M + p.NT * 8 - 1) / (p.NT * 8);
    if (p.TB < 1) p.TB = 1;
    p.RB = (N + 127) / 128;
    p.KS = K / 16;
    int ks_cap = kGemmSmemCap / (p.NT * 512);
    int smin = (p.KS + ks_cap - 1) / ks_cap;
    int best = smin;
    double best_score = -1.0;
    for (int s = smin; s <= 32 && s <= p.KS; ++s) {
        if (s > smin && p.KS / s < 8) break;
        long ctas = (long)p.RB * s * p.TB;
        long waves = (ctas + kWaveCtas - 1) / kWaveCtas;
        double eff = (double)ctas / (double)(waves * kWaveCtas);
        double score = eff - 0.004 * s;   // each extra slice costs partial-sum traffic
        if (score > best_score) { best_score = score; best = s; }
    }
    p.S = best;
    int ksl = (p.KS + p.S - 1) / p.S + 1;
    p.smem = (size_t)ksl * p.NT * 512;
    return p;
}

// Repack row-major bf16 W[N][K] into MMA A-fragment order:
// packed[(rt*KS + ks)*32 + lane] = { W[r][c], W[r][c+1] | W[r+8][c], W[r+8][c+1] |
//                                    W[r][c+8], W[r][c+9] | W[r+8][c+8], W[r+8][c+9] }
// with r = rt*16 + lane/4, c = ks*16 + 2*(lane%4).
__global__ void gemm_pack_kernel(const uint16_t* __restrict__ W, uint4* __restrict__ packed, int N, int K) {
    const int KS = K / 16;
    const size_t total = (size_t)(N / 16) * KS * 32;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int lane = (int)(i & 31);
        size_t tile = i >> 5;
        int ks = (int)(tile % KS);
        int rt = (int)(tile / KS);
        int r = rt * 16 + (lane >> 2), c = ks * 16 + 2 * (lane & 3);
        const uint16_t* w0 = W + (size_t)r * K + c;
        const uint16_t* w1 = W + (size_t)(r + 8) * K + c;
        uint4 v;
        v.x = pack2(w0[0], w0[1]);
        v.y = pack2(w1[0], w1[1]);
        v.z = pack2(w0[8], w0[9]);
        v.w = pack2(w1[8], w1[9]);
        packed[i] = v;
    }
}

struct GemmArgs {
    const uint4* W;   // packed weights
    const float* x;   // [M][ldx]
    float* out;       // [S][M][N] partial sums (S == 1: the result itself)
    int M, N, K, ldx;
    int S, KS;
};

template <int NT>
__global__ void __launch_bounds__(kGemmThreads, 2) gemm_wstream_kernel(GemmArgs a) {
    extern __shared__ uint4 Bs[];  // [ks_local][NT][32 lanes] = {hi.b0, hi.b1, lo.b0, lo.b1}
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int rb = blockIdx.x / a.S, s = blockIdx.x % a.S;
    const int tok0 = blockIdx.y * (NT * 8);
    const int ks0 = (int)(((long)a.KS * s) / a.S), ks1 = (int)(((long)a.KS * (s + 1)) / a.S);
    const int nks = ks1 - ks0;
    const int rt = rb * 8 + warp;
    const bool active = rt * 16 < a.N;

    // Issue the first weight loads before staging the activations: they do not depend on them.
    const uint4* wp = a.W + ((size_t)rt * a.KS + ks0) * 32 + lane;
    uint4 buf[kGemmDepth];
#pragma unroll
    for (int i = 0; i < kGemmDepth; ++i)
        if (active && i < nks) buf[i] = ldg_stream(wp + (size_t)i * 32);

    // Stage x[tok0 .. tok0+NT*8)[ks0*16 .. ks1*16) as split-bf16 B fragments.
    for (int idx = threadIdx.x; idx < nks * NT * 32; idx += kGemmThreads) {
        int l = idx & 31, nt = (idx >> 5) % NT, ksl = idx / (32 * NT);
        int tok = tok0 + nt * 8 + (l >> 2);
        int k = (ks0 + ksl) * 16 + 2 * (l & 3);
        float2 v0 = make_float2(0.f, 0.f), v1 = make_float2(0.f, 0.f);
        if (tok < a.M) {
            const float* xr = a.x + (size_t)tok * a.ldx + k;
            v0 = *reinterpret_cast<const float2*>(xr);
            v1 = *reinterpret_cast<const float2*>(xr + 8);
        }
        uint16_t h0, l0, h1, l1, h2, l2, h3, l3;
        split_bf16(v0.x, h0, l0); split_bf16(v0.y, h1, l1);
        split_bf16(v1.x, h2, l2); split_bf16(v1.y, h3, l3);
        Bs[idx] = make_uint4(pack2(h0, h1), pack2(h2, h3), pack2(l0, l1), pack2(l2, l3));
    }
    __syncthreads();
    if (!active) return;

    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[nt][j] = 0.f;

    for (int base = 0; base < nks; base += kGemmDepth) {
#pragma unroll
        for (int i = 0; i < kGemmDepth; ++i) {
            int ks = base + i;
            if (ks < nks) {
                uint4 af = buf[i];
                if (ks + kGemmDepth < nks) buf[i] = ldg_stream(wp + (size_t)(ks + kGemmDepth) * 32);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    uint4 b = Bs[(ks * NT + nt) * 32 + lane];
                    mma_bf16_16816(acc[nt], af, b.x, b.y);
                    mma_bf16_16816(acc[nt], af, b.z, b.w);
                }
            }
        }
    }

    // C fragment: c0,c1 -> (row g, tokens 2t, 2t+1); c2,c3 -> (row g+8, same tokens).
    float* outp = a.out + (size_t)s * a.M * a.N;
    const int r0 = rt * 16 + g;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        int tok = tok0 + nt * 8 + 2 * t;
        if (tok < a.M) {
            outp[(size_t)tok * a.N + r0] = acc[nt][0];
            outp[(size_t)tok * a.N + r0 + 8] = acc[nt][2];
        }
        if (tok + 1 < a.M) {
            outp[(size_t)(tok + 1) * a.N + r0] = acc[nt][1];
            outp[(size_t)(tok + 1) * a.N + r0 + 8] = acc[nt][3];
        }
    }
}

// y[i] = sum_s part[s][i], fixed order.
__global__ void reduce_partials_kernel(const float* __restrict__ part, float* __restrict__ y, size_t n, int S) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float v = 0.f;
        for (int s = 0; s < S; ++s) v += part[(size_t)s * n + i];
        y[i] = v;
    }
}

static inline cudaError_t gemm_launch(const GemmPlan& p, const uint4* W, const float* x, int ldx, float* out,
                                      int M, int N, int K, cudaStream_t st) {
    GemmArgs a{W, x, out, M, N, K, ldx, p.S, p.KS};
    dim3 grid(p.RB * p.S, p.TB);
    switch (p.NT) {
        case 1: gemm_wstream_kernel<1><<<grid, kGemmThreads, p.smem, st>>>(a); break;
        case 2: gemm_wstream_kernel<2><<<grid, kGemmThreads, p.smem, st>>>(a); break;
        case 3: gemm_wstream_kernel<3><<<grid, kGemmThreads, p.smem, st>>>(a); break;
        default: gemm_wstream_kernel<4><<<grid, kGemmThreads, p.smem, st>>>(a); break;
    }
    return cudaGetLastError();
}

static inline cudaError_t gemm_init_attrs() {
    cudaError_t e;
    e = cudaFuncSetAttribute(gemm_wstream_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemCap + 4096);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_wstream_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemCap + 4096);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_wstream_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemCap + 4096);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(gemm_wstream_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemCap + 4096);
}

}  // namespace pipesd
