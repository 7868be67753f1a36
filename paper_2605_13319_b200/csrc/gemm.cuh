// Small-M weight-streaming GEMM: y[M,N] = x[M,K] . W[N,K]^T, bf16 W (read once from HBM), fp32 x.
//
// The weight matrix is the wide operand: a 16-row x 16-column tile of W is the A fragment of a
// warp-level m16n8k16 MMA and the (few) token rows are the narrow N dimension.  W is repacked once
// at context creation into fragment order, 4 KB per (128-row block, k16 step), so that a chunk of
// consecutive k-steps of a row block is one contiguous run in HBM.
// One producer lane streams those runs into a shared-memory ring with bulk asynchronous copies
// (cp.async.bulk + mbarrier transaction counts); four consumer warps, two row tiles each, read their
// fragments back with conflict-free 16-byte loads and issue the MMAs.  The ring is the kernel's
// memory-level parallelism: up to three CTAs x 3-4 stages x 16 KB are in flight per SM, and because
// weights do not depend on the previous kernel, the ring is filled BEFORE the programmatic-dependent-
// launch wait, so the weight stream of kernel n+1 starts while kernel n is still draining.
// Activations stay fp32 in the residual stream; the kernels that produce a GEMM input store it
// already split into bf16 hi + lo terms in B-fragment order ("xf" arrays), so the matching chunk of
// activations rides in the same ring stage as its weights (two MMAs, one fp32 accumulator: 2^-17).
// Work split: CTA = (128-row block of W, K slice, token block); partial sums of the K slices go to a
// scratch array [S][M][N] that the consuming kernel adds up in fixed order (deterministic).
#pragma once
#include "common.cuh"

namespace pipesd {

constexpr int kGemmConsumerWarps = 4;                       // x 2 row tiles x 16 rows = 128 rows per CTA
constexpr int kGemmThreads = (kGemmConsumerWarps + 1) * 32;  // + one producer warp
constexpr int kGemmKC = 4;                                   // k16 steps per ring stage
constexpr int kGemmWStage = kGemmKC * 4096;                  // weight bytes per stage
constexpr int kGemmCtasPerSm = 3;
constexpr int kGemmWave = 148 * kGemmCtasPerSm;

__host__ __device__ constexpr int gemm_stages(int NT) { return NT == 1 ? 4 : 3; }
__host__ __device__ constexpr int gemm_stage_bytes(int NT) { return kGemmWStage + kGemmKC * NT * 512; }
__host__ __device__ constexpr int gemm_smem_bytes(int NT) { return gemm_stages(NT) * gemm_stage_bytes(NT) + 128; }

struct GemmPlan {
    int NT;  // n8 token tiles per token block (1..4)
    int TB;  // token blocks
    int RB;  // 128-row blocks
    int S;   // K slices
    int KS;  // k16 steps in K
};

// Tiles per token block / token blocks for M rows: shared by the GEMM and by the producers of xf arrays.
__host__ __device__ inline int xf_nt(int M) { int nt = (M + 7) / 8; return nt > 4 ? 4 : (nt < 1 ? 1 : nt); }
__host__ __device__ inline int xf_tb(int M) { int nt = xf_nt(M); return (M + nt * 8 - 1) / (nt * 8); }
// uint4 elements of the xf array of an [M, K] activation.
__host__ __device__ inline size_t xf_elems(int M, int K) { return (size_t)xf_tb(M) * (K / 16) * xf_nt(M) * 32; }

static int g_gemm_force_split = 0;   // 0: choose automatically (tuning hook)

// Host: choose the K split.  CTAs are small and three fit on an SM, so what matters is a grid of a few
// waves whose last wave is nearly full, against the partial-sum traffic every extra slice adds.
static inline GemmPlan gemm_plan(int M, int N, int K) {
    GemmPlan p;
    p.NT = xf_nt(M);
    p.TB = xf_tb(M);
    p.RB = (N + 127) / 128;
    p.KS = K / 16;
    int best = 1;
    double best_score = -1e9;
    const int mrows = M < p.NT * 8 ? M : p.NT * 8;
    for (int s = 1; s <= 64 && s <= p.KS; ++s) {
        if (s > 1 && p.KS / s < 2 * kGemmKC) break;
        long ctas = (long)p.RB * s * p.TB;
        long waves = (ctas + kGemmWave - 1) / kGemmWave;
        double eff = (double)ctas / (double)(waves * kGemmWave);
        double partial = s > 1 ? 4.0 * s * mrows / (double)K : 0.0;   // partial bytes (w+r) / weight bytes
        double score = eff - 0.5 * partial;
        if (score > best_score) { best_score = score; best = s; }
    }
    p.S = g_gemm_force_split > 0 && g_gemm_force_split <= p.KS ? g_gemm_force_split : best;
    return p;
}

// Bytes of the packed copy of W[N][K] (row blocks padded to 128 rows).
static inline size_t gemm_packed_bytes(int N, int K) { return (size_t)((N + 127) / 128) * 128 * K * 2; }

// Repack row-major bf16 W rows [0, n_rows) into MMA A-fragment order, starting at packed row row0:
// packed[((rb*KS + ks)*8 + tile)*32 + lane] = { W[r][c], W[r][c+1] | W[r+8][c], W[r+8][c+1] |
//                                               W[r][c+8], W[r][c+9] | W[r+8][c+8], W[r+8][c+9] }
// with r = (rb*8 + tile)*16 + lane/4 (in packed-row numbering), c = ks*16 + 2*(lane%4).
// Rows beyond the source (padding of the last row block) are zero.  row0 and n_rows: multiples of 16.
__global__ void gemm_pack_kernel(const uint16_t* __restrict__ W, uint4* __restrict__ packed, int row0, int n_rows,
                                 int K, int pad_to) {
    const int KS = K / 16;
    const int rt0 = row0 / 16, n_rt = (pad_to - row0) / 16;
    const size_t total = (size_t)n_rt * KS * 32;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int lane = (int)(i & 31);
        size_t tile = i >> 5;
        int ks = (int)(tile % KS);
        int rt = rt0 + (int)(tile / KS);
        int r = (rt - rt0) * 16 + (lane >> 2), c = ks * 16 + 2 * (lane & 3);
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (r < n_rows) {
            const uint16_t* w0 = W + (size_t)r * K + c;
            const uint16_t* w1 = W + (size_t)(r + 8) * K + c;
            v.x = pack2(w0[0], w0[1]);
            v.y = pack2(w1[0], w1[1]);
            v.z = pack2(w0[8], w0[9]);
            v.w = pack2(w1[8], w1[9]);
        }
        int rb = rt >> 3, tl = rt & 7;
        packed[(((size_t)rb * KS + ks) * 8 + tl) * 32 + lane] = v;
    }
}

// fp32 x[M][K] -> xf (split-bf16 B fragments).  One thread per (token, even k).
__global__ void xf_format_kernel(const float* __restrict__ x, uint32_t* __restrict__ xf, int M, int K) {
    const int KS = K / 16, NT = xf_nt(M);
    size_t n = (size_t)M * (K / 2);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        int tok = (int)(i / (K / 2)), k = 2 * (int)(i % (K / 2));
        float2 v = *reinterpret_cast<const float2*>(x + (size_t)tok * K + k);
        xf_store_pair(xf, tok, k, v.x, v.y, KS, NT);
    }
}

struct GemmArgs {
    const uint4* W;    // packed weights
    const uint4* xf;   // activations, split-bf16 B fragments [tb][ks][nt][32]
    float* out;        // [S][M][N] partial sums (S == 1: the result itself)
    int* err;          // device error word (nullable): set when a bounded wait gives up
    int M, N, S, KS;
};

template <int NT>
__global__ void __launch_bounds__(kGemmThreads, kGemmCtasPerSm) gemm_wstream_kernel(GemmArgs a) {
    constexpr int kStages = gemm_stages(NT);
    constexpr int kStageBytes = gemm_stage_bytes(NT);
    constexpr int kBStage = kGemmKC * NT * 512;
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);   // full[kStages], empty[kStages]
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kStages;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rb = blockIdx.x / a.S, s = blockIdx.x % a.S, tb = blockIdx.y;
    const int ks0 = (int)(((long)a.KS * s) / a.S), ks1 = (int)(((long)a.KS * (s + 1)) / a.S);
    const int nks = ks1 - ks0, nchunks = (nks + kGemmKC - 1) / kGemmKC;

    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < kStages; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, kGemmConsumerWarps);
        }
        fence_mbar_init();
    }
    __syncthreads();
    pdl_launch_dependents();

    if (warp == kGemmConsumerWarps) {
        // ---------------- producer: one lane streams (weights, activations) chunks into the ring
        if (lane == 0) {
            const unsigned char* wsrc = reinterpret_cast<const unsigned char*>(a.W) + ((size_t)rb * a.KS + ks0) * 4096;
            const unsigned char* bsrc =
                reinterpret_cast<const unsigned char*>(a.xf) + ((size_t)tb * a.KS + ks0) * (NT * 512);
            auto chunk_ks = [&](int c) { int r = nks - c * kGemmKC; return r < kGemmKC ? r : kGemmKC; };
            const int pre = nchunks < kStages ? nchunks : kStages;
            // weights do not depend on the previous kernel: start them before the dependency wait
            for (int c = 0; c < pre; ++c) {
                const int kc = chunk_ks(c);
                mbar_expect_tx(full0 + 8 * c, (uint32_t)kc * (4096 + NT * 512));
                bulk_g2s(smem_base + c * kStageBytes, wsrc + (size_t)c * kGemmWStage, (uint32_t)kc * 4096, full0 + 8 * c);
            }
            pdl_wait();
            for (int c = 0; c < pre; ++c) {
                const int kc = chunk_ks(c);
                bulk_g2s(smem_base + c * kStageBytes + kGemmWStage, bsrc + (size_t)c * kBStage, (uint32_t)kc * NT * 512,
                         full0 + 8 * c);
            }
            bool ok = true;
            int issued = pre;
            for (int c = pre; c < nchunks && ok; ++c) {
                const int st = c % kStages, kc = chunk_ks(c);
                ok = mbar_wait(empty0 + 8 * st, ((c / kStages) - 1) & 1);
                if (!ok) break;
                mbar_expect_tx(full0 + 8 * st, (uint32_t)kc * (4096 + NT * 512));
                bulk_g2s(smem_base + st * kStageBytes, wsrc + (size_t)c * kGemmWStage, (uint32_t)kc * 4096, full0 + 8 * st);
                bulk_g2s(smem_base + st * kStageBytes + kGemmWStage, bsrc + (size_t)c * kBStage,
                         (uint32_t)kc * NT * 512, full0 + 8 * st);
                issued = c + 1;
            }
            if (!ok) {
                if (a.err) atomicExch(a.err, 1);
                // give up: let every copy already issued land before this CTA's shared memory is released
                for (int c = issued > kStages ? issued - kStages : 0; c < issued; ++c)
                    mbar_wait(full0 + 8 * (c % kStages), (c / kStages) & 1);
            }
        }
        return;
    }

    // ---------------- consumers: warp w owns row tiles 2w and 2w+1 of the block
    float acc[2][NT][4];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[j][nt][e] = 0.f;

    bool ok = true;
    for (int c = 0; c < nchunks; ++c) {
        const int st = c % kStages;
        ok = mbar_wait(full0 + 8 * st, (c / kStages) & 1);
        if (!ok) break;
        const unsigned char* wst = smem + st * kStageBytes;
        const unsigned char* bst = wst + kGemmWStage;
        int kc = nks - c * kGemmKC;
        kc = kc < kGemmKC ? kc : kGemmKC;
#pragma unroll
        for (int k = 0; k < kGemmKC; ++k) {
            if (k < kc) {
                const uint4 a0 = *reinterpret_cast<const uint4*>(wst + ((k * 8 + warp * 2) * 32 + lane) * 16);
                const uint4 a1 = *reinterpret_cast<const uint4*>(wst + ((k * 8 + warp * 2 + 1) * 32 + lane) * 16);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint4 b = *reinterpret_cast<const uint4*>(bst + ((k * NT + nt) * 32 + lane) * 16);
                    mma_bf16_16816(acc[0][nt], a0, b.x, b.y);
                    mma_bf16_16816(acc[1][nt], a1, b.x, b.y);
                    mma_bf16_16816(acc[0][nt], a0, b.z, b.w);
                    mma_bf16_16816(acc[1][nt], a1, b.z, b.w);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * st);
    }
    if (!ok) {
        if (a.err && lane == 0) atomicExch(a.err, 2);
        return;
    }

    // C fragment: c0,c1 -> (row g, tokens 2t, 2t+1); c2,c3 -> (row g+8, same tokens).
    const int g = lane >> 2, t = lane & 3;
    float* outp = a.out + (size_t)s * a.M * a.N;
    const int tok0 = tb * (NT * 8);
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int r0 = ((rb * 8 + warp * 2 + j) * 16) + g;
        if (r0 >= a.N) continue;      // padding rows of the last block (N is a multiple of 16)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int tok = tok0 + nt * 8 + 2 * t;
            if (tok < a.M) {
                outp[(size_t)tok * a.N + r0] = acc[j][nt][0];
                outp[(size_t)tok * a.N + r0 + 8] = acc[j][nt][2];
            }
            if (tok + 1 < a.M) {
                outp[(size_t)(tok + 1) * a.N + r0] = acc[j][nt][1];
                outp[(size_t)(tok + 1) * a.N + r0 + 8] = acc[j][nt][3];
            }
        }
    }
}

// y[i] = sum_s part[s][i], fixed order.
__global__ void reduce_partials_kernel(const float* __restrict__ part, float* __restrict__ y, size_t n, int S) {
    pdl_wait();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float v = 0.f;
        for (int s = 0; s < S; ++s) v += part[(size_t)s * n + i];
        y[i] = v;
    }
}

static inline cudaError_t gemm_launch(const GemmPlan& p, const uint4* W, const uint4* xf, float* out, int* err,
                                      int M, int N, cudaStream_t st) {
    GemmArgs a{W, xf, out, err, M, N, p.S, p.KS};
    dim3 grid(p.RB * p.S, p.TB);
    switch (p.NT) {
        case 1: return launch_pdl(gemm_wstream_kernel<1>, grid, dim3(kGemmThreads), gemm_smem_bytes(1), st, a);
        case 2: return launch_pdl(gemm_wstream_kernel<2>, grid, dim3(kGemmThreads), gemm_smem_bytes(2), st, a);
        case 3: return launch_pdl(gemm_wstream_kernel<3>, grid, dim3(kGemmThreads), gemm_smem_bytes(3), st, a);
        default: return launch_pdl(gemm_wstream_kernel<4>, grid, dim3(kGemmThreads), gemm_smem_bytes(4), st, a);
    }
}

template <typename K>
static inline cudaError_t gemm_set_attr(K kernel, int NT) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, gemm_smem_bytes(NT));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
}

static inline cudaError_t gemm_init_attrs() {
    cudaError_t e;
    if ((e = gemm_set_attr(gemm_wstream_kernel<1>, 1)) != cudaSuccess) return e;
    if ((e = gemm_set_attr(gemm_wstream_kernel<2>, 2)) != cudaSuccess) return e;
    if ((e = gemm_set_attr(gemm_wstream_kernel<3>, 3)) != cudaSuccess) return e;
    return gemm_set_attr(gemm_wstream_kernel<4>, 4);
}

}  // namespace pipesd
