// Small-M weight-streaming GEMM with fused epilogues: y[M,N] = x[M,K] . W[N,K]^T, bf16 W (read once
// from HBM), fp32 x.
//
// The weight matrix is the wide operand: a 16-row x 16-column tile of W is the A fragment of a
// warp-level m16n8k16 MMA and the (few) token rows are the narrow N dimension.  W is repacked once
// at context creation into fragment order, 4 KB per (128-row block, k16 step), so that a chunk of
// consecutive k-steps of a row block is one contiguous run in HBM.
// One producer lane streams those runs into a shared-memory ring with bulk asynchronous copies
// (cp.async.bulk + mbarrier transaction counts); four consumer warps, two row tiles each, read their
// fragments back with conflict-free 16-byte loads and issue the MMAs.  The ring is the kernel's
// memory-level parallelism, and because weights do not depend on the previous kernel it is filled
// BEFORE the programmatic-dependent-launch wait: the weight stream of kernel n+1 starts while kernel n
// is still draining.
// Activations stay fp32 in the residual stream; the kernel that produces a GEMM input stores it already
// split into bf16 hi + lo terms in B-fragment order ("xf" arrays), so the matching chunk of activations
// rides in the same ring stage as its weights (two MMAs, one fp32 accumulator: 2^-17 relative).
// Split-K: the S CTAs that share a row block form a thread-block cluster.  Each of the block's eight 16-row tiles
// is owned by one rank; every CTA writes its partial tiles straight into their owners' shared memory (remote
// stores over distributed shared memory, posted), one cluster barrier follows, and each owner sums what it
// received in rank order (deterministic) and runs the epilogue -- no partial sums in global memory, no remote
// loads, and nobody has to wait for anybody after the barrier.
// Epilogues: plain fp32 output; RoPE + q store + bf16 K/V page append (QKV); residual add + next RMSNorm's
// gain and sum of squares (O and down projections); SiLU(gate)*up (gate/up projection).  RMSNorm itself
// never runs as a kernel: the producer stores x*gain and per-block sums of squares, the consumer scales
// its result rows by rsqrt(mean(x^2)+eps), which commutes with the matrix product.
#pragma once
#include "common.cuh"

namespace pipesd {

constexpr int kGemmConsumerWarps = 4;                       // x 2 row tiles x 16 rows = 128 rows per CTA
constexpr int kGemmConsumers = kGemmConsumerWarps * 32;
constexpr int kGemmThreads = kGemmConsumers + 32;           // + one producer warp
constexpr int kGemmKC = 4;                                  // k16 steps per ring stage
constexpr int kGemmWStage = kGemmKC * 4096;                 // weight bytes per stage
constexpr int kGemmMinStages = 2, kGemmMaxStages = 6;
constexpr int kGemmCtasPerSm = 3;
constexpr int kGemmWave = 148 * kGemmCtasPerSm;
constexpr int kGemmMaxSplit = 8;                            // portable cluster size
constexpr int kGemmSmemTail = 128 + 128 + 1024;             // barriers | rstd[32] | tile sums of squares [8][32]

enum GemmMode { kPlain = 0, kQkvRope = 1, kResid = 2, kSwiglu = 3 };


__host__ __device__ constexpr int gemm_stage_bytes(int NT) { return kGemmWStage + kGemmKC * NT * 512; }
// partial tiles received from the cluster: [owned tile][source rank][token][16 rows] fp32
__host__ __device__ constexpr int gemm_recv_bytes(int NT, int S) { return ((8 + S - 1) / S) * S * (NT * 8) * 64; }
__host__ __device__ constexpr int gemm_smem_bytes(int NT, int stages, int S) {
    return stages * gemm_stage_bytes(NT) + kGemmSmemTail + gemm_recv_bytes(NT, S);
}

struct GemmPlan {
    int NT;  // n8 token tiles per token block (1..4)
    int TB;  // token blocks
    int RB;  // 128-row blocks
    int S;   // K slices = cluster size
    int KS;  // k16 steps in K
    int stages;  // ring depth
};

// Tiles per token block / token blocks for M rows: shared by the GEMM and by the producers of xf arrays.
__host__ __device__ inline int xf_nt(int M) { int nt = (M + 7) / 8; return nt > 4 ? 4 : (nt < 1 ? 1 : nt); }
__host__ __device__ inline int xf_tb(int M) { int nt = xf_nt(M); return (M + nt * 8 - 1) / (nt * 8); }
// uint4 elements of the xf array of an [M, K] activation.
__host__ __device__ inline size_t xf_elems(int M, int K) { return (size_t)xf_tb(M) * (K / 16) * xf_nt(M) * 32; }

// Host: choose the K split (cluster size).  What matters is enough CTAs to keep ~100 KB of copies in
// flight per SM and a last wave that is nearly full.
static inline GemmPlan gemm_plan(int M, int N, int K) {
    GemmPlan p;
    p.NT = xf_nt(M);
    p.TB = xf_tb(M);
    p.RB = (N + 127) / 128;
    p.KS = K / 16;
    // One resident wave if possible: every CTA streams from the first microsecond and the next kernel's
    // CTAs find room to prefetch.  Largest K split that still fits the wave of a single token block.  The
    // split depends on (N, K) only, never on M: the order in which a result element is summed is then the
    // same whether a request is verified alone or inside a batch (bit-identical decisions).
    int best = 1;
    for (int s = 1; s <= kGemmMaxSplit && s <= p.KS; ++s) {
        if (s > 1 && p.KS / s < 2 * kGemmKC) break;
        if ((long)p.RB * s <= kGemmWave) best = s;
    }
    p.S = best;
    // ring depth: as deep as the shared memory of an SM allows for the number of CTAs it will hold.  A clustered
    // GEMM always leaves room for three CTAs per SM, even when it brings fewer: at two 113 KB CTAs per SM a B200
    // holds exactly the 32 clusters of eight that the O and down projections launch, so one foreign CTA in a GPC
    // pushed a cluster into a second wave, and the next kernel's CTAs found no room to start and prefetch their
    // weights under this kernel's tail.  Three stages instead of five for those two: -0.14 ms per 7B pass at up to 16
    // rows.  With three or four token tiles per block the MMA work per chunk is 1.5-2x and the deeper ring wins
    // (7b, 17 rows: 3.81 ms with five stages, 4.00 ms with three), so those keep the depth by CTA count.
    long ctas = (long)p.RB * p.S * p.TB;
    int per_sm = (int)((ctas + 147) / 148);
    if (p.S > 1 && p.NT <= 2) per_sm = kGemmCtasPerSm;
    per_sm = per_sm < 1 ? 1 : (per_sm > kGemmCtasPerSm ? kGemmCtasPerSm : per_sm);
    int budget = (227 * 1024) / per_sm - 1024 - kGemmSmemTail - gemm_recv_bytes(p.NT, p.S);
    p.stages = budget / gemm_stage_bytes(p.NT);
    p.stages = p.stages < kGemmMinStages ? kGemmMinStages : (p.stages > kGemmMaxStages ? kGemmMaxStages : p.stages);
    return p;
}

// Bytes of the packed copy of W[N][K] (row blocks padded to 128 rows).
static inline size_t gemm_packed_bytes(int N, int K) { return (size_t)((N + 127) / 128) * 128 * K * 2; }

// ---- packed-row <-> logical-row maps of the fused layouts ------------------------------------------
// QKV: inside every head, tile tau holds dims 8*tau..8*tau+7 in rows 0..7 and their rotary partners
// (+hd/2) in rows 8..15, so that one thread owns both elements of a rotation pair.
__host__ __device__ inline int qkv_logical_row(int packed_row, int hd) {
    const int head = packed_row / hd, within = packed_row % hd, tau = within >> 4, i = within & 15;
    return head * hd + (i < 8 ? 8 * tau + i : hd / 2 + 8 * tau + (i - 8));
}
// gate/up: tile rows 0..7 are gate features f..f+7, rows 8..15 the matching up features.
__host__ __device__ inline int gu_feature(int packed_row) { return (packed_row >> 4) * 8 + (packed_row & 7); }

struct PackSrc {
    const uint16_t* w[3];   // up to three row-major [rows_i][K] sources, concatenated along N
    int rows[3];
    int mode;               // GemmMode of the consumer (row permutation)
    int hd;                 // head width (kQkvRope)
};

// Repack into MMA A-fragment order: packed[((rb*KS + ks)*8 + tile)*32 + lane] =
//   { W[r][c], W[r][c+1] | W[r+8][c], W[r+8][c+1] | W[r][c+8], W[r][c+9] | W[r+8][c+8], W[r+8][c+9] }
// with r = (rb*8 + tile)*16 + lane/4 in packed-row numbering, c = ks*16 + 2*(lane%4); packed rows map to
// logical rows per `mode`; rows beyond the sources (padding of the last row block) are zero.
__global__ void gemm_pack_kernel(PackSrc src, uint4* __restrict__ packed, int n_rows, int K) {
    const int KS = K / 16;
    const int n_rt = (n_rows + 127) / 128 * 8;
    const size_t total = (size_t)n_rt * KS * 32;
    auto fetch = [&](int pr, int c, uint32_t& lo, uint32_t& hi) {
        lo = hi = 0u;
        if (pr >= n_rows) return;
        int lr, which = 0;
        if (src.mode == kSwiglu) { which = (pr & 15) < 8 ? 0 : 1; lr = gu_feature(pr); }
        else {
            lr = src.mode == kQkvRope ? qkv_logical_row(pr, src.hd) : pr;
            while (which < 2 && lr >= src.rows[which]) { lr -= src.rows[which]; ++which; }
        }
        const uint16_t* w = src.w[which] + (size_t)lr * K + c;
        lo = pack2(w[0], w[1]);
        hi = pack2(w[8], w[9]);
    };
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int lane = (int)(i & 31);
        const size_t tile = i >> 5;
        const int ks = (int)(tile % KS), rt = (int)(tile / KS);
        const int r = rt * 16 + (lane >> 2), c = ks * 16 + 2 * (lane & 3);
        uint4 v;
        fetch(r, c, v.x, v.z);
        fetch(r + 8, c, v.y, v.w);
        packed[(((size_t)(rt >> 3) * KS + ks) * 8 + (rt & 7)) * 32 + lane] = v;
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
    const uint4* W;     // packed weights
    const uint4* xf;    // activations, split-bf16 B fragments [tb][ks][nt][32]
    int* err;           // device error word (nullable): set when a bounded wait gives up
    int M, N, S, KS, stages;
    // input normalisation (nullable): ssq_in[b*M + tok], b < n_ssq, are sums of squares of the un-normalised
    // input row; the result rows are scaled by rsqrt(sum / d_in + eps)
    const float* ssq_in;
    int n_ssq, d_in;
    float eps;
    // kPlain
    float* out;         // [M][N]
    // kQkvRope
    float* q_out;       // [M][Hq*hd] rotated queries
    uint16_t* kv_pool;
    const float* cs;    // [M][hd/2] cos / sin of the row's position
    const float* sn;
    const long long* row_kvoff;   // [M] element offset of the row's K row inside a layer (head 0, column 0)
    int Hq, Hkv, hd, layer, n_pages, page_size;
    // kResid
    float* x;           // residual stream [M][N], updated in place
    uint16_t* xf_out;   // x_new * gain_next as split-bf16 fragments (K of the consumer = N)
    const float* gain_next;
    float* ssq_out;     // [RB][M] sums of squares of x_new over the row block's columns
    // kSwiglu
    uint16_t* xf_act;   // silu(gate)*up as split-bf16 fragments, feature-major K = N/2
    // the successor's weights this kernel pulls into L2 once its own last chunk has been requested
    L2Prefetch pf;
};

// Host: the L2 hint that covers `depth_bytes` of every CTA's weight range of the GEMM (M, N, K) over `W`, after the
// chunks that GEMM's CTAs copy by themselves before their dependency wait (their whole ring).
static inline L2Prefetch gemm_prefetch_of(const void* W, int M, int N, int K, uint32_t depth_bytes) {
    L2Prefetch pf = {};
    if (W == nullptr || depth_bytes == 0) return pf;
    const GemmPlan p = gemm_plan(M, N, K);
    const uint32_t run = (uint32_t)(p.KS / p.S) * 4096u;           // K slices differ by at most one k16 step: a hint may be off by that
    const uint32_t skip = (uint32_t)p.stages * kGemmWStage;
    if (run <= skip) return pf;
    pf.ptr = reinterpret_cast<const unsigned char*>(W);
    pf.run_bytes = run;
    pf.skip = skip;
    pf.len = run - skip < depth_bytes ? run - skip : depth_bytes;
    pf.runs = p.RB * p.S;
    return pf;
}

template <int NT, int MODE>
__global__ void __launch_bounds__(kGemmThreads, kGemmCtasPerSm) gemm_wstream_kernel(const GemmArgs a) {
    constexpr int kStageBytes = gemm_stage_bytes(NT);
    constexpr int kBStage = kGemmKC * NT * 512;
    constexpr int MT = NT * 8;                        // tokens per token block
    extern __shared__ __align__(128) unsigned char smem[];
    const int stages = a.stages;
    unsigned char* tail = smem + stages * kStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);              // full[stages], empty[stages]
    float* rstd_s = reinterpret_cast<float*>(tail + 128);             // [32]
    float* tss_s = rstd_s + 32;                                       // rank 0: [8 tiles][32 tokens] sums of squares of the new rows
    float* recv = reinterpret_cast<float*>(tail + kGemmSmemTail);     // [owned tile][source rank][token MT][row 16]
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kGemmMaxStages;
    const uint32_t ssq_bar = full0 + 8 * 2 * kGemmMaxStages;           // rank 0: one arrival per rank once its tile sums are stored
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rb = blockIdx.x / a.S, s = blockIdx.x % a.S, tb = blockIdx.y;   // s == rank in the cluster
    const int ks0 = (int)(((long)a.KS * s) / a.S), ks1 = (int)(((long)a.KS * (s + 1)) / a.S);
    const int nks = ks1 - ks0, nchunks = (nks + kGemmKC - 1) / kGemmKC;
    const int tok0 = tb * MT;

    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, kGemmConsumerWarps);
        }
        if (MODE == kResid) mbar_init(ssq_bar, (uint32_t)a.S);
        fence_mbar_init();
    }
    __syncthreads();
    pdl_launch_dependents();

    // epilogue inputs that live in global memory are fetched right after the dependency wait, long before the
    // epilogue needs them (only when a rank owns at most two tiles, i.e. S >= 4)
    const bool prefetch = (8 + a.S - 1) / a.S <= 2;
    float pf_a[2][NT], pf_b[2][NT], pf_g[2];
    long long pf_kv[NT];

    bool ok = true;
    if (warp == kGemmConsumerWarps) {
        // ---------------- producer warp: lane 0 streams (weights, activations) chunks into the ring
        if (lane == 0) {
            const unsigned char* wsrc = reinterpret_cast<const unsigned char*>(a.W) + ((size_t)rb * a.KS + ks0) * 4096;
            const unsigned char* bsrc =
                reinterpret_cast<const unsigned char*>(a.xf) + ((size_t)tb * a.KS + ks0) * (NT * 512);
            auto chunk_ks = [&](int c) { int r = nks - c * kGemmKC; return r < kGemmKC ? r : kGemmKC; };
            const int pre = nchunks < stages ? nchunks : stages;
            const uint64_t pol = l2_evict_first_policy();   // weights are read once: they must not push the activations out of L2
            // weights do not depend on the previous kernel: start them before the dependency wait
            for (int c = 0; c < pre; ++c) {
                const int kc = chunk_ks(c);
                mbar_expect_tx(full0 + 8 * c, (uint32_t)kc * (4096 + NT * 512));
                bulk_g2s_hint(smem_base + c * kStageBytes, wsrc + (size_t)c * kGemmWStage, (uint32_t)kc * 4096, full0 + 8 * c, pol);
            }
            pdl_wait();
            for (int c = 0; c < pre; ++c) {
                const int kc = chunk_ks(c);
                bulk_g2s(smem_base + c * kStageBytes + kGemmWStage, bsrc + (size_t)c * kBStage, (uint32_t)kc * NT * 512,
                         full0 + 8 * c);
            }
            int issued = pre, st = 0;
            uint32_t ph = 0;                       // parity of the empty-barrier phase being waited for
            for (int c = pre; c < nchunks; ++c) {
                const int kc = chunk_ks(c);
                ok = mbar_wait(empty0 + 8 * st, ph);
                if (!ok) break;
                mbar_expect_tx(full0 + 8 * st, (uint32_t)kc * (4096 + NT * 512));
                bulk_g2s_hint(smem_base + st * kStageBytes, wsrc + (size_t)c * kGemmWStage, (uint32_t)kc * 4096, full0 + 8 * st, pol);
                bulk_g2s(smem_base + st * kStageBytes + kGemmWStage, bsrc + (size_t)c * kBStage,
                         (uint32_t)kc * NT * 512, full0 + 8 * st);
                issued = c + 1;
                if (++st == stages) { st = 0; ph ^= 1u; }
            }
            if (!ok) {
                if (a.err) atomicExch(a.err, 1);
                // give up: let every copy already issued land before this CTA's shared memory is released
                for (int c = issued > stages ? issued - stages : 0; c < issued; ++c)
                    mbar_wait(full0 + 8 * (c % stages), (c / stages) & 1);
            }
        } else if (a.ssq_in != nullptr) {
            // lanes 1..31: the input's RMSNorm factor per token (off the critical path)
            pdl_wait();
            for (int tl = lane - 1; tl < MT; tl += 31) {
                const int tok = tok0 + tl;
                float ss = 0.f;
                if (tok < a.M) {
                    for (int b0 = 0; b0 < a.n_ssq; b0 += 32) {
                        float part[32];
#pragma unroll
                        for (int b = 0; b < 32; ++b)     // all loads of a batch in flight together
                            part[b] = b0 + b < a.n_ssq ? a.ssq_in[(size_t)(b0 + b) * a.M + tok] : 0.f;
#pragma unroll
                        for (int b = 0; b < 32; ++b) ss += part[b];
                    }
                }
                rstd_s[tl] = rsqrtf(ss / (float)a.d_in + a.eps);
            }
        }
        __syncwarp();
    } else {
        // ---------------- consumers: warp w owns row tiles 2w and 2w+1 of the block
        if ((MODE == kResid || MODE == kQkvRope) && prefetch) {
            pdl_wait();
            const int row = threadIdx.x & 15, tg = threadIdx.x >> 4;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int tile = s + q * a.S, pr = rb * 128 + tile * 16 + row;
                pf_g[q] = 0.f;
#pragma unroll
                for (int i = 0; i < NT; ++i) {
                    const int tok = tok0 + tg + 8 * i;
                    pf_a[q][i] = pf_b[q][i] = 0.f;
                    if (tile < 8 && tok < a.M && pr < a.N) {
                        if (MODE == kResid) {
                            pf_a[q][i] = a.x[(size_t)tok * a.N + pr];
                        } else {
                            const int half = a.hd / 2, dim = qkv_logical_row(pr, a.hd) % a.hd;
                            pf_a[q][i] = a.cs[(size_t)tok * half + (dim % half)];
                            pf_b[q][i] = a.sn[(size_t)tok * half + (dim % half)];
                        }
                    }
                }
                if (MODE == kResid && tile < 8 && pr < a.N) pf_g[q] = a.gain_next[pr];
            }
            if (MODE == kQkvRope) {
#pragma unroll
                for (int i = 0; i < NT; ++i) {
                    const int tok = tok0 + tg + 8 * i;
                    pf_kv[i] = tok < a.M ? a.row_kvoff[tok] : 0;
                }
            }
        }
        float acc[2][NT][4];
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[j][nt][e] = 0.f;

        int st = 0;
        uint32_t ph = 0;
        for (int c = 0; c < nchunks; ++c) {
            ok = mbar_wait(full0 + 8 * st, ph);
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
            if (++st == stages) { st = 0; ph ^= 1u; }
        }
        if (!ok && a.err && lane == 0) atomicExch(a.err, 2);
        // this CTA has consumed its last weights: from here on HBM idles until the successor streams
        if (ok) l2_prefetch_issue(a.pf, (int)(blockIdx.y * gridDim.x + blockIdx.x), (int)(gridDim.x * gridDim.y), threadIdx.x, kGemmConsumers);
        // Every partial tile goes to the rank that owns the tile (tile % S), into slot [tile / S][this rank] of its receive
        // buffer: token-major rows of 16 floats, as the epilogue reads them.
        const int g = lane >> 2, t = lane & 3;
        const uint32_t recv_a = smem_u32(recv);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int tile = warp * 2 + j, owner = tile % a.S, q = tile / a.S;
            const uint32_t slot = recv_a + (uint32_t)((q * a.S + s) * MT * 64);
            const uint32_t dst = a.S > 1 ? dsmem_addr(slot, (uint32_t)owner) : slot;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const uint32_t pt = dst + (uint32_t)((nt * 8 + 2 * t) * 64);
                if (a.S > 1) {
                    dsmem_st_f32(pt + g * 4, acc[j][nt][0]);
                    dsmem_st_f32(pt + 64 + g * 4, acc[j][nt][1]);
                    dsmem_st_f32(pt + (g + 8) * 4, acc[j][nt][2]);
                    dsmem_st_f32(pt + 64 + (g + 8) * 4, acc[j][nt][3]);
                } else {
                    float* pl = recv + ((q * a.S + s) * MT + nt * 8 + 2 * t) * 16;
                    pl[g] = acc[j][nt][0];
                    pl[16 + g] = acc[j][nt][1];
                    pl[g + 8] = acc[j][nt][2];
                    pl[16 + g + 8] = acc[j][nt][3];
                }
            }
        }
    }

    // ---------------- cluster reduction + epilogue (all 160 threads reach the barrier, also on errors): after it every
    // partial of this CTA's tiles has arrived, and nobody writes to or reads from another CTA's shared memory any more
    if (a.S > 1) cluster_sync_all(); else __syncthreads();
    pdl_wait();   // (long satisfied) every thread that touches the predecessors' global data has waited itself
    if (warp < kGemmConsumerWarps) {
        const int row = threadIdx.x & 15, tg = threadIdx.x >> 4;   // 16 lanes = the 16 rows of a tile
        // One tile of the row block: sum the S partial tiles in rank order, then the mode's epilogue.
        // xin / gin / cin / sin_ : prefetched epilogue inputs of this tile, or null to load them here.
        auto epi_tile = [&](int tile, const float* xin, const float* gin, const float* cin, const float* sin_) {
            const int pr = rb * 128 + tile * 16 + row;               // packed row
            float pv[NT][kGemmMaxSplit];
            const float* rt = recv + (size_t)(tile / a.S) * a.S * MT * 16;    // this tile's partials, one per source rank
#pragma unroll
            for (int i = 0; i < NT; ++i) {
#pragma unroll
                for (int r = 0; r < kGemmMaxSplit; ++r)
                    pv[i][r] = r < a.S ? rt[(r * MT + tg + 8 * i) * 16 + row] : 0.f;
            }
#pragma unroll
            for (int i = 0; i < NT; ++i) {
                const int tl = tg + 8 * i, tok = tok0 + tl;
                float v = 0.f;
#pragma unroll
                for (int r = 0; r < kGemmMaxSplit; ++r) v += pv[i][r];
                if (a.ssq_in != nullptr) v *= rstd_s[tl];
                const bool live = tok < a.M && pr < a.N;
                if (MODE == kPlain) {
                    if (live) a.out[(size_t)tok * a.N + pr] = v;
                } else if (MODE == kResid) {
                    float xn = 0.f;
                    if (live) {
                        float* xp = a.x + (size_t)tok * a.N + pr;
                        xn = (xin ? xin[i] : *xp) + v;
                        *xp = xn;
                        xf_store_one(a.xf_out, tok, pr, xn * (gin ? gin[0] : a.gain_next[pr]), a.N / 16, NT);
                    }
                    // sum of squares over the tile's 16 rows (lanes of a half-warp), fixed order
                    float q = xn * xn;
                    q += __shfl_xor_sync(0xffffffffu, q, 1);
                    q += __shfl_xor_sync(0xffffffffu, q, 2);
                    q += __shfl_xor_sync(0xffffffffu, q, 4);
                    q += __shfl_xor_sync(0xffffffffu, q, 8);
                    if (row == 0) {
                        // tile sums go to rank 0's shared memory, which adds the 8 tiles up once every rank has reported
                        const uint32_t dst = smem_u32(tss_s + tile * 32 + tl);
                        if (a.S > 1) dsmem_st_f32(dsmem_addr(dst, 0u), q); else tss_s[tile * 32 + tl] = q;
                    }
                } else {
                    // both remaining modes pair row i (< 8) with row i + 8 of the tile
                    const float partner = __shfl_xor_sync(0xffffffffu, v, 8);
                    if (MODE == kSwiglu) {
                        if (row < 8 && live) {
                            const float act = v / (1.f + expf(-v)) * partner;      // own = gate, partner = up
                            xf_store_one(a.xf_act, tok, gu_feature(pr), act, (a.N / 2) / 16, NT);
                        }
                    } else if (live) {                                           // kQkvRope
                        const int lr = qkv_logical_row(pr, a.hd);                 // head * hd + dim
                        const int head = lr / a.hd, dim = lr % a.hd, half = a.hd / 2;
                        float val = v;
                        if (head < a.Hq + a.Hkv) {                                // q and k heads are rotated
                            const float c = cin ? cin[i] : a.cs[(size_t)tok * half + (dim % half)];
                            const float sgn = sin_ ? sin_[i] : a.sn[(size_t)tok * half + (dim % half)];
                            val = row < 8 ? v * c - partner * sgn : v * c + partner * sgn;
                        }
                        if (head < a.Hq) {
                            a.q_out[((size_t)tok * a.Hq + head) * a.hd + dim] = val;
                        } else {
                            const int kv = head < a.Hq + a.Hkv ? 0 : 1;
                            const int kvh = kv ? head - a.Hq - a.Hkv : head - a.Hq;
                            const size_t per_head = (size_t)a.page_size * a.hd;
                            const long long rk = cin ? pf_kv[i] : a.row_kvoff[tok];   // the row's offset inside a layer (head 0, K)
                            const size_t off = (size_t)a.layer * a.n_pages * 2 * a.Hkv * per_head + (size_t)rk +
                                               ((size_t)kv * a.Hkv + kvh) * per_head + kv_col_offset(dim);
                            a.kv_pool[off] = f32_to_bf16_bits(val);
                        }
                    }
                }
            }
        };
        if (prefetch) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int tile = s + q * a.S;
                if (tile < 8) epi_tile(tile, pf_a[q], &pf_g[q], pf_a[q], pf_b[q]);
            }
        } else {
            for (int tile = s; tile < 8; tile += a.S) epi_tile(tile, nullptr, nullptr, nullptr, nullptr);
        }
        if (MODE == kResid) {
            // Sums of squares of the new rows: every rank has stored its tiles' sums in rank 0's shared memory; one
            // thread per rank reports that (a release that covers the CTA's stores through the barrier before it) and the
            // rank is done.  Rank 0 waits for the S reports, adds the eight tiles up in order and writes the block's sum.
            asm volatile("bar.sync 1, %0;" ::"n"(kGemmConsumers) : "memory");
            if (threadIdx.x == 0) {
                if (a.S > 1)
                    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(dsmem_addr(ssq_bar, 0u)) : "memory");
                else
                    mbar_arrive(ssq_bar);
            }
            if (s == 0 && threadIdx.x < 32) {
                bool got = false;
                for (uint32_t it = 0; it < (1u << 22) && !got; ++it) {
                    uint32_t okw;
                    asm volatile(
                        "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                        : "=r"(okw) : "r"(ssq_bar), "r"(0u) : "memory");
                    got = okw != 0;
                }
                if (!got && a.err && threadIdx.x == 0) atomicExch(a.err, 5);
                for (int tl = threadIdx.x; tl < MT; tl += 32) {
                    const int tok = tok0 + tl;
                    if (tok < a.M) {
                        float q = 0.f;
#pragma unroll
                        for (int tile = 0; tile < 8; ++tile) q += tss_s[tile * 32 + tl];
                        a.ssq_out[(size_t)rb * a.M + tok] = got ? q : 0.f;
                    }
                }
            }
        }
    }
}

template <int MODE>
static inline cudaError_t gemm_launch_mode(const GemmPlan& p, const GemmArgs& a, cudaStream_t st) {
    dim3 grid(p.RB * p.S, p.TB);
    switch (p.NT) {
        case 1: return launch_pdl_cluster(gemm_wstream_kernel<1, MODE>, grid, dim3(kGemmThreads), gemm_smem_bytes(1, p.stages, p.S), st, p.S, a);
        case 2: return launch_pdl_cluster(gemm_wstream_kernel<2, MODE>, grid, dim3(kGemmThreads), gemm_smem_bytes(2, p.stages, p.S), st, p.S, a);
        case 3: return launch_pdl_cluster(gemm_wstream_kernel<3, MODE>, grid, dim3(kGemmThreads), gemm_smem_bytes(3, p.stages, p.S), st, p.S, a);
        default: return launch_pdl_cluster(gemm_wstream_kernel<4, MODE>, grid, dim3(kGemmThreads), gemm_smem_bytes(4, p.stages, p.S), st, p.S, a);
    }
}

static inline cudaError_t gemm_launch(int mode, const GemmPlan& p, GemmArgs a, cudaStream_t st) {
    a.S = p.S;
    a.KS = p.KS;
    a.stages = p.stages;
    switch (mode) {
        case kQkvRope: return gemm_launch_mode<kQkvRope>(p, a, st);
        case kResid: return gemm_launch_mode<kResid>(p, a, st);
        case kSwiglu: return gemm_launch_mode<kSwiglu>(p, a, st);
        default: return gemm_launch_mode<kPlain>(p, a, st);
    }
}

template <int NT, int MODE>
static inline cudaError_t gemm_set_attr() {
    cudaError_t e = cudaFuncSetAttribute(gemm_wstream_kernel<NT, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         gemm_smem_bytes(NT, kGemmMaxStages, 7));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(gemm_wstream_kernel<NT, MODE>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
}
template <int MODE>
static inline cudaError_t gemm_set_attr_mode() {
    cudaError_t e;
    if ((e = gemm_set_attr<1, MODE>()) != cudaSuccess) return e;
    if ((e = gemm_set_attr<2, MODE>()) != cudaSuccess) return e;
    if ((e = gemm_set_attr<3, MODE>()) != cudaSuccess) return e;
    return gemm_set_attr<4, MODE>();
}
static inline cudaError_t gemm_init_attrs() {
    cudaError_t e;
    if ((e = gemm_set_attr_mode<kPlain>()) != cudaSuccess) return e;
    if ((e = gemm_set_attr_mode<kQkvRope>()) != cudaSuccess) return e;
    if ((e = gemm_set_attr_mode<kResid>()) != cudaSuccess) return e;
    return gemm_set_attr_mode<kSwiglu>();
}

}  // namespace pipesd
