// Persistent layer-stack kernel for small token counts (M <= 32 rows): the weight stream never stops.
//
// One CTA per SM stays resident for a whole sequence of GEMM "phases" (O projection, gate/up, down, the next
// layer's QKV, ... , LM head).  Every phase is cut into 256-row units x chunks of 4 k16-steps, and the
// flattened (unit, chunk) list is dealt out in equal contiguous ranges to the CTAs ("stream-K"), so that all
// SMs stream the same number of weight bytes whatever the matrix shape.  Inside a CTA
//   - a weight-producer thread walks the CTA's chunk list of ALL phases and keeps a 5-6 stage shared-memory
//     ring (32 KB of packed weights per stage) full with bulk asynchronous copies; weights depend on nothing,
//     so the stream runs ahead across phase boundaries for as long as the ring has room;
//   - an activation-producer warp waits until the phase that produces the input has finished everywhere (a
//     counter in global memory, released by the epilogues), then adds the matching activation fragments to
//     the stages and, where the phase normalises its input, derives the rows' RMSNorm factors;
//   - eight consumer warps (2 row tiles each) run the warp-level MMAs (bf16 weights x split-bf16 activations,
//     fp32 accumulate) and the fused epilogues straight from their accumulator fragments.
// A unit whose chunks are spread over several CTAs is summed through global memory: every contributor
// stores its accumulator fragments, takes a ticket, and the last one to arrive adds all contributions in
// CTA order (a fixed order: the result does not depend on who arrived last) and runs the epilogue.  Nobody
// waits for anybody except at the phase boundary, and that wait is hidden behind the weights already
// prefetched for the next phase.  Every wait is bounded; a wait that gives up raises the device error word,
// which every other wait polls, so that the kernel always terminates.
#pragma once
#include "common.cuh"
#include "gemm.cuh"

namespace pipesd {

constexpr int kMegaConsumerWarps = 8;
constexpr int kMegaConsumers = kMegaConsumerWarps * 32;
constexpr int kMegaThreads = kMegaConsumers + 64;          // + weight-producer warp + activation-producer warp
constexpr int kMegaKC = 4;                                 // k16 steps per chunk
constexpr int kMegaWHalf = kMegaKC * 4096;                 // one 128-row block of a chunk
constexpr int kMegaWStage = 2 * kMegaWHalf;                // 256 rows
constexpr int kMegaMaxStages = 6;
constexpr int kMegaTail = 2048;                            // barriers | rstd[32] | ssq exchange [8][32] | flag
constexpr int kMegaMaxCtas = 160;
constexpr int kMegaSmemMax = 227 * 1024;
constexpr unsigned long long kMegaWaitNs = 1000000000ull;  // bound of every wait

__host__ __device__ constexpr int mega_stage_bytes(int NT) { return kMegaWStage + kMegaKC * NT * 512; }
__host__ __device__ constexpr int mega_stages(int NT) {
    return (kMegaSmemMax - kMegaTail) / mega_stage_bytes(NT) > kMegaMaxStages ? kMegaMaxStages
                                                                               : (kMegaSmemMax - kMegaTail) / mega_stage_bytes(NT);
}
__host__ __device__ constexpr int mega_smem_bytes(int NT) { return mega_stages(NT) * mega_stage_bytes(NT) + kMegaTail; }

// One GEMM of the chain.  Built once per context; lives in device memory.
struct MegaPhase {
    const uint4* W;        // packed weights (128-row blocks in MMA A-fragment order)
    const uint4* xf;       // input activations, split-bf16 B fragments of one token block
    int mode;              // GemmMode
    int N, KS, RB;         // logical rows, k16 steps, 128-row blocks
    int UB, CPR, T;        // 256-row units, chunks per unit, chunks in the phase
    int ticket0;           // first ticket counter of the phase
    const float* ssq_in;   // sums of squares of the un-normalised input rows [n_ssq][M] (null: no input norm)
    int n_ssq;
    int layer;             // kQkvRope
    float* out;            // kPlain [M][N]
    float* x;              // kResid: residual stream [M][N]
    uint16_t* xf_out;      // kResid: x_new * gain_next as fragments;  kSwiglu: silu(gate)*up as fragments
    const float* gain_next;
    float* ssq_out;        // kResid: [UB][M]
};

struct MegaArgs {
    const MegaPhase* phases;
    int p0, p1;            // phase range of this launch
    int launch_idx;        // position of this launch in the pass
    int M;
    int* done;             // [n_phases] finished units per phase (zero at the start of a pass)
    int* tickets;          // per (phase, unit) arrival counters (zero at the start of a pass)
    int* arrived;          // CTAs of this launch that have started
    float4* scratch;       // accumulator fragments of partial units: [cta][2][2*NT][256]
    int* err;              // device error word
    float eps;
    int d_in;
    // kQkvRope
    float* q_out;
    uint16_t* kv_pool;
    const float* cs;
    const float* sn;
    const long long* row_kvoff;
    int Hq, Hkv, hd, n_pages, page_size;
};

__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_relaxed(const int* p) {
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(int* p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

#ifdef PIPESD_MEGA_TRACE
// Development build only: per (launch, phase, CTA) timestamps of the phase-boundary anatomy.
__device__ unsigned long long g_mega_trace[64 * 4 * kMegaMaxCtas * 8];
#define MEGA_TRACE(k)                                                                                          \
    do {                                                                                                        \
        if (a.launch_idx < 64)                                                                                  \
            g_mega_trace[(((size_t)a.launch_idx * 4 + (p - a.p0)) * kMegaMaxCtas + cta) * 8 + (k)] = global_ns(); \
    } while (0)
#else
#define MEGA_TRACE(k) do { } while (0)
#endif

// mbarrier wait that also gives up when another part of the grid has raised the error word.
__device__ __forceinline__ bool mbar_wait_err(uint32_t bar, uint32_t parity, const int* err) {
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((it & 255u) == 255u) {
            if (ld_relaxed(err) != 0) return false;
            const uint64_t now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kMegaWaitNs) return false;
        }
    }
}
// Wait until *ctr >= target (acquire).
__device__ __forceinline__ bool poll_counter(const int* ctr, int target, const int* err) {
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (ld_acquire(ctr) >= target) return true;
        if ((it & 63u) == 63u) {
            if (ld_relaxed(err) != 0) return false;
            const uint64_t now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kMegaWaitNs) return false;
        }
    }
}

// CTA that owns chunk c when T chunks are dealt to G CTAs as [floor(T*i/G), floor(T*(i+1)/G)).
__device__ __forceinline__ int mega_owner(int c, int T, int G) { return (int)((((long long)c + 1) * G - 1) / T); }
__device__ __forceinline__ int mega_begin(int i, int T, int G) { return (int)(((long long)T * i) / G); }

__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

constexpr int kMegaL2Ahead = 8;   // chunks (of 32 KB) a blocked weight producer pulls into L2 beyond its ring

// Cursor over one CTA's weight chunks through the phases of a launch.
struct MegaWalk {
    int p, p1, c, ce, u, cc, KS, CPR, RB;
    const unsigned char* W;
    __device__ __forceinline__ void load_phase(const MegaArgs& a, int cta, int G) {
        for (; p < p1; ++p) {
            const MegaPhase& ph = a.phases[p];
            c = mega_begin(cta, ph.T, G);
            ce = mega_begin(cta + 1, ph.T, G);
            if (c < ce) {
                KS = ph.KS; CPR = ph.CPR; RB = ph.RB;
                W = reinterpret_cast<const unsigned char*>(ph.W);
                u = c / CPR;
                cc = c - u * CPR;
                return;
            }
        }
    }
    __device__ __forceinline__ void start(const MegaArgs& a, int cta, int G) { p = a.p0; p1 = a.p1; load_phase(a, cta, G); }
    __device__ __forceinline__ bool valid() const { return p < p1; }
    __device__ __forceinline__ void next(const MegaArgs& a, int cta, int G) {
        if (++c < ce) { if (++cc == CPR) { cc = 0; ++u; } return; }
        ++p;
        load_phase(a, cta, G);
    }
    __device__ __forceinline__ int kc() const { const int ks = cc * kMegaKC; return KS - ks < kMegaKC ? KS - ks : kMegaKC; }
    __device__ __forceinline__ bool two() const { return 2 * u + 1 < RB; }
    __device__ __forceinline__ const unsigned char* src(int half) const {
        return W + ((size_t)(2 * u + half) * KS + cc * kMegaKC) * 4096;
    }
    __device__ __forceinline__ void prefetch_l2() const {
        const uint32_t bytes = (uint32_t)kc() * 4096u;
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src(0)), "r"(bytes) : "memory");
        if (two()) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src(1)), "r"(bytes) : "memory");
    }
};

// Stores one token tile of an xf array from the epilogue's fragment layout.  Thread (g, t) holds, for tokens
// 2t and 2t+1 of tile nt (index b), the values of k = 16*ks + g (h = 0) and k = 16*ks + g + 8 (h = 1).  A B
// fragment wants k = 2t', 2t'+1, 2t'+8, 2t'+9 of one token in one 16-byte word: the two threads of a pair
// g = 2t', 2t'+1 (lanes 4 apart) swap one token each, then the even one stores token 2t, the odd one 2t+1.
// All 32 lanes must call this (shuffles); `M` masks padding tokens.
__device__ __forceinline__ void xf_store_frag(uint4* xf, int ks, int nt, int NT, int g, int t, const float (&v)[2][2],
                                              int M, bool rows_live) {
    const bool odd = g & 1;
    const float s0 = odd ? v[0][0] : v[1][0], s1 = odd ? v[0][1] : v[1][1];     // the partner's token
    const float r0 = __shfl_xor_sync(0xffffffffu, s0, 4), r1 = __shfl_xor_sync(0xffffffffu, s1, 4);
    const int b = odd ? 1 : 0;
    const float e0 = odd ? r0 : v[b][0], o0 = odd ? v[b][0] : r0;               // k even / odd, h = 0
    const float e1 = odd ? r1 : v[b][1], o1 = odd ? v[b][1] : r1;               // h = 1
    uint32_t h0, l0, h1, l1;
    {
        uint16_t ha, la, hb, lb;
        split_bf16(e0, ha, la); split_bf16(o0, hb, lb);
        h0 = pack2(ha, hb); l0 = pack2(la, lb);
        split_bf16(e1, ha, la); split_bf16(o1, hb, lb);
        h1 = pack2(ha, hb); l1 = pack2(la, lb);
    }
    const int tok = nt * 8 + 2 * t + b;
    if (rows_live && tok < M) xf[((size_t)ks * NT + nt) * 32 + (2 * t + b) * 4 + (g >> 1)] = make_uint4(h0, h1, l0, l1);
}

// Epilogue of one finished 256-row unit from accumulator fragments: thread (warp, lane = 4g + t) holds, for
// row tile 2*warp + j and token tile nt, rows g (e = 0, 1) and g + 8 (e = 2, 3) of tokens 2t and 2t + 1.
// The fused layouts put a rotary pair / a (gate, up) pair in rows g and g + 8 of one tile: both in one thread.
template <int NT, int MODE>
__device__ __forceinline__ void mega_epilogue(const MegaArgs& a, const MegaPhase& ph, int u, int warp, int lane,
                                              float (&acc)[2][NT][4], const float* rstd_s, float* ssq_w) {
    const int g = lane >> 2, t = lane & 3;
    const int N = ph.N;
    if (ph.ssq_in != nullptr) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const float r0 = rstd_s[nt * 8 + 2 * t], r1 = rstd_s[nt * 8 + 2 * t + 1];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                acc[j][nt][0] *= r0; acc[j][nt][2] *= r0;
                acc[j][nt][1] *= r1; acc[j][nt][3] *= r1;
            }
        }
    }
    if (MODE == kResid) {
        float ssq_loc[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) ssq_loc[nt][0] = ssq_loc[nt][1] = 0.f;
        float xv[2][NT][4];
        // all loads of the residual stream first, then the updates
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int pr = u * 256 + (2 * warp + j) * 16 + g;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int tok = nt * 8 + 2 * t + (e & 1);
                    xv[j][nt][e] = (pr < N && tok < a.M) ? __ldcg(ph.x + (size_t)tok * N + pr + 8 * (e >> 1)) : 0.f;
                }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int pr = u * 256 + (2 * warp + j) * 16 + g;
            const bool row_live = pr < N;
            float gain_lo = 0.f, gain_hi = 0.f;
            if (row_live) { gain_lo = ph.gain_next[pr]; gain_hi = ph.gain_next[pr + 8]; }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float v[2][2];
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    const int tok = nt * 8 + 2 * t + b;
                    const float xlo = xv[j][nt][b] + acc[j][nt][b], xhi = xv[j][nt][2 + b] + acc[j][nt][2 + b];
                    if (row_live && tok < a.M) {
                        float* xp = ph.x + (size_t)tok * N + pr;
                        xp[0] = xlo;
                        xp[8] = xhi;
                        ssq_loc[nt][b] += xlo * xlo + xhi * xhi;
                    }
                    v[b][0] = xlo * gain_lo;
                    v[b][1] = xhi * gain_hi;
                }
                xf_store_frag(reinterpret_cast<uint4*>(ph.xf_out), u * 16 + 2 * warp + j, nt, NT, g, t, v, a.M, row_live);
            }
        }
        // sums of squares of the unit's 256 rows per token: over the 8 row groups of a warp by shuffles,
        // over the 8 warps through shared memory, both in a fixed order
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                float v = ssq_loc[nt][b];
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                v += __shfl_xor_sync(0xffffffffu, v, 8);
                v += __shfl_xor_sync(0xffffffffu, v, 16);
                if (g == 0) ssq_w[warp * 32 + nt * 8 + 2 * t + b] = v;
            }
        asm volatile("bar.sync 1, %0;" ::"n"(kMegaConsumers) : "memory");
        const int tok = threadIdx.x;
        if (tok < NT * 8 && tok < a.M) {
            float q = 0.f;
#pragma unroll
            for (int w = 0; w < kMegaConsumerWarps; ++w) q += ssq_w[w * 32 + tok];
            ph.ssq_out[(size_t)u * a.M + tok] = q;
        }
        return;
    }
    if (MODE == kSwiglu) {
        // rows g: gate, g + 8: up of feature (pr >> 4) * 8 + g; tiles j = 0, 1 of a warp are the two halves
        // (k and k + 8) of one k16 step of the down projection's input
        const bool row_live = u * 256 + (2 * warp + 1) * 16 + g < N;      // N is a multiple of 32 rows here
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float v[2][2];
#pragma unroll
            for (int b = 0; b < 2; ++b)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const float gt = acc[j][nt][b], up = acc[j][nt][2 + b];
                    v[b][j] = gt / (1.f + expf(-gt)) * up;
                }
            xf_store_frag(reinterpret_cast<uint4*>(ph.xf_out), u * 8 + warp, nt, NT, g, t, v, a.M, row_live);
        }
        return;
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int pr = u * 256 + (2 * warp + j) * 16 + g;      // packed rows pr and pr + 8
        if (pr >= N) continue;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                const int tok = nt * 8 + 2 * t + b;
                const float vlo = acc[j][nt][b], vhi = acc[j][nt][2 + b];
                if (tok >= a.M) continue;
                if (MODE == kPlain) {
                    float* o = ph.out + (size_t)tok * N + pr;
                    o[0] = vlo;
                    o[8] = vhi;
                } else {                                                        // kQkvRope
                    const int head = pr / a.hd, within = pr - head * a.hd, half = a.hd / 2;
                    const int dim = 8 * (within >> 4) + g;                      // rows g / g+8 <-> dims dim / dim+half
                    float olo = vlo, ohi = vhi;
                    if (head < a.Hq + a.Hkv) {
                        const float c = a.cs[(size_t)tok * half + dim], s = a.sn[(size_t)tok * half + dim];
                        olo = vlo * c - vhi * s;
                        ohi = vhi * c + vlo * s;
                    }
                    if (head < a.Hq) {
                        float* qp = a.q_out + ((size_t)tok * a.Hq + head) * a.hd + dim;
                        qp[0] = olo;
                        qp[half] = ohi;
                    } else {
                        const int kv = head < a.Hq + a.Hkv ? 0 : 1;
                        const int kvh = kv ? head - a.Hq - a.Hkv : head - a.Hq;
                        const size_t per_head = (size_t)a.page_size * a.hd;
                        uint16_t* kp = a.kv_pool + (size_t)ph.layer * a.n_pages * 2 * a.Hkv * per_head +
                                       (size_t)a.row_kvoff[tok] + ((size_t)kv * a.Hkv + kvh) * per_head + dim;
                        kp[0] = f32_to_bf16_bits(olo);
                        kp[half] = f32_to_bf16_bits(ohi);
                    }
                }
            }
        }
    }
}

template <int NT>
__global__ void __launch_bounds__(kMegaThreads, 1) mega_kernel(const MegaArgs a) {
    constexpr int kStage = mega_stage_bytes(NT);
    constexpr int kStages = mega_stages(NT);
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* tail = smem + kStages * kStage;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);          // fullW[8] | fullX[8] | empty[8]
    float* rstd_s = reinterpret_cast<float*>(tail + 256);        // [32]
    float* ssq_w = reinterpret_cast<float*>(tail + 512);         // [8][32]
    int* flag_s = reinterpret_cast<int*>(tail + 512 + 1024);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t fullW0 = smem_u32(bars), fullX0 = fullW0 + 64, empty0 = fullW0 + 128;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = (int)gridDim.x, cta = (int)blockIdx.x;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(fullW0 + 8 * i, 1);
            mbar_init(fullX0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, kMegaConsumerWarps);
        }
        fence_mbar_init();
        red_release_add(a.arrived, 1);
    }
    __syncthreads();

    if (warp == kMegaConsumerWarps) {
        // ------------------------------------------------ weight producer: runs ahead of everything
        if (lane != 0) return;
        MegaWalk ring, pf;               // next chunk for the ring / next chunk to prefetch into L2
        ring.start(a, cta, G);
        pf = ring;
        int n = 0, st = 0, n_pf = 0;
        bool ok = true;
        while (ring.valid()) {
            if (n >= kStages) {
                // Ring full: the consumers are held up (usually at a phase boundary).  HBM must not go idle
                // meanwhile: pull the chunks after the ring's into L2, up to kMegaL2Ahead chunks ahead.
                const uint32_t bar = empty0 + 8 * st, par = (uint32_t)((n / kStages) - 1) & 1u;
                uint64_t t0 = 0;
                for (uint32_t it = 0; !mbar_try(bar, par); ++it) {
                    if (n_pf < n + kMegaL2Ahead && pf.valid()) {
                        if (n_pf >= n) pf.prefetch_l2();
                        pf.next(a, cta, G);
                        ++n_pf;
                        continue;
                    }
                    if ((it & 255u) == 255u) {
                        if (ld_relaxed(a.err) != 0) { ok = false; break; }
                        const uint64_t now = global_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > kMegaWaitNs) { ok = false; break; }
                    }
                }
                if (!ok) break;
            }
            const uint32_t bytes = (uint32_t)ring.kc() * 4096u;
            const bool two = ring.two();
            mbar_expect_tx(fullW0 + 8 * st, two ? 2 * bytes : bytes);
            bulk_g2s(smem_base + st * kStage, ring.src(0), bytes, fullW0 + 8 * st);
            if (two) bulk_g2s(smem_base + st * kStage + kMegaWHalf, ring.src(1), bytes, fullW0 + 8 * st);
            if (++st == kStages) st = 0;
            ring.next(a, cta, G);
            ++n;
        }
        if (!ok) {
            atomicCAS(a.err, 0, 11);
            // let every copy already issued land before the CTA's shared memory can be released
            for (int i = n > kStages ? n - kStages : 0; i < n; ++i)
                mbar_wait(fullW0 + 8 * (i % kStages), (uint32_t)(i / kStages) & 1u);
        }
        return;
    }

    if (warp == kMegaConsumerWarps + 1) {
        // ------------------------------------------------ activation producer
        int n = 0, st = 0;
        bool ok = true;
        for (int p = a.p0; p < a.p1; ++p) {
            const MegaPhase& ph = a.phases[p];
            if (p == a.p0) {
                pdl_wait();                       // the kernels launched before this one have completed
            } else {
                if (lane == 0) ok = poll_counter(a.done + (p - 1), a.phases[p - 1].UB, a.err);
                ok = __shfl_sync(0xffffffffu, ok, 0);
            }
            if (!ok) break;
            if (lane == 0) MEGA_TRACE(0);
            if (p == a.p1 - 1) {
                // Successor kernels may be scheduled from here on -- but only once every CTA of this grid
                // is resident: a successor that took the place of a CTA still to come would wait for this
                // grid while this grid's phase boundaries wait for that CTA.
                if (lane == 0) ok = poll_counter(a.arrived, G, a.err);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                pdl_launch_dependents();
            }
            const int T = ph.T, CPR = ph.CPR, KS = ph.KS;
            const int cb = mega_begin(cta, T, G), ce = mega_begin(cta + 1, T, G);
            if (cb == ce) continue;
            if (ph.ssq_in != nullptr && lane < NT * 8) {
                float ss = 0.f;
                if (lane < a.M)
                    for (int b = 0; b < ph.n_ssq; ++b) ss += __ldcg(ph.ssq_in + (size_t)b * a.M + lane);
                rstd_s[lane] = rsqrtf(ss / (float)a.d_in + a.eps);
            }
            __syncwarp();
            if (lane == 0) {
                fence_proxy_async_all();          // activations were written with ordinary stores by other SMs
                const unsigned char* X = reinterpret_cast<const unsigned char*>(ph.xf);
                int cc = cb % CPR;
                for (int c = cb; c < ce; ++c, ++n) {
                    if (n >= kStages) {
                        ok = mbar_wait_err(empty0 + 8 * st, (uint32_t)((n / kStages) - 1) & 1u, a.err);
                        if (!ok) break;
                    }
                    const int ks = cc * kMegaKC;
                    const int kc = KS - ks < kMegaKC ? KS - ks : kMegaKC;
                    const uint32_t bytes = (uint32_t)kc * NT * 512u;
                    mbar_expect_tx(fullX0 + 8 * st, bytes);
                    bulk_g2s(smem_base + st * kStage + kMegaWStage, X + (size_t)ks * NT * 512, bytes, fullX0 + 8 * st);
                    if (++st == kStages) st = 0;
                    if (++cc == CPR) cc = 0;
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            n = __shfl_sync(0xffffffffu, n, 0);
            st = __shfl_sync(0xffffffffu, st, 0);
            if (!ok) break;
        }
        if (!ok && lane == 0) {
            atomicCAS(a.err, 0, 12);
            for (int i = n > kStages ? n - kStages : 0; i < n; ++i)
                mbar_wait(fullX0 + 8 * (i % kStages), (uint32_t)(i / kStages) & 1u);
        }
        return;
    }

    // ---------------------------------------------------- consumers: warp w owns row tiles 2w, 2w+1 of a unit
    pdl_wait();      // epilogues read what earlier kernels wrote (rotary tables, K/V offsets, residual stream)
    int n = 0, st = 0;
    bool ok = true;
    const unsigned w_off = (unsigned)(warp >> 2) * kMegaWHalf + (unsigned)((warp & 3) * 2 * 32 + lane) * 16;
    for (int p = a.p0; p < a.p1; ++p) {
        const MegaPhase& ph = a.phases[p];
        const int T = ph.T, CPR = ph.CPR, KS = ph.KS, RB = ph.RB, mode = ph.mode;
        const int cb = mega_begin(cta, T, G), ce = mega_begin(cta + 1, T, G);
        int c = cb;
        while (c < ce) {
            const int u = c / CPR, ub = u * CPR;
            const int se = ce < ub + CPR ? ce : ub + CPR;
            const bool has_rows = 2 * u + (warp >> 2) < RB;     // a last unit may hold one 128-row block only
            float acc[2][NT][4];
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[j][nt][e] = 0.f;
            for (; c < se; ++c, ++n) {
                // A wait that gave up is not an exit: the warp keeps walking the schedule (without waiting or
                // computing) so that it still meets the other consumer warps at every named barrier below.
                if (ok) {
                    const uint32_t par = (uint32_t)(n / kStages) & 1u;
                    ok = mbar_wait_err(fullW0 + 8 * st, par, a.err) && mbar_wait_err(fullX0 + 8 * st, par, a.err);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok && lane == 0) atomicCAS(a.err, 0, 13);
                }
                if (ok) {
                    const unsigned char* wst = smem + st * kStage + w_off;
                    const unsigned char* bst = smem + st * kStage + kMegaWStage + lane * 16;
                    const int ks = (c - ub) * kMegaKC;
                    const int kc = KS - ks < kMegaKC ? KS - ks : kMegaKC;
                    if (has_rows) {
#pragma unroll
                        for (int k = 0; k < kMegaKC; ++k) {
                            if (k < kc) {
                                const uint4 a0 = *reinterpret_cast<const uint4*>(wst + k * 4096);
                                const uint4 a1 = *reinterpret_cast<const uint4*>(wst + k * 4096 + 512);
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) {
                                    const uint4 b = *reinterpret_cast<const uint4*>(bst + (k * NT + nt) * 512);
                                    mma_bf16_16816(acc[0][nt], a0, b.x, b.y);
                                    mma_bf16_16816(acc[1][nt], a1, b.x, b.y);
                                    mma_bf16_16816(acc[0][nt], a0, b.z, b.w);
                                    mma_bf16_16816(acc[1][nt], a1, b.z, b.w);
                                }
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty0 + 8 * st);
                    if (threadIdx.x == 0 && c == cb) MEGA_TRACE(1);
                }
                if (++st == kStages) st = 0;
            }
            if (threadIdx.x == 0) MEGA_TRACE(2);
            // ---- the CTA's part of unit u is summed.  Alone on the unit: epilogue.  Otherwise leave the
            // fragments in global memory; the last contributor to arrive sums all of them in CTA order.
            const int i0 = mega_owner(ub, T, G), i1 = mega_owner(ub + CPR - 1, T, G);
            if (i0 != i1) {
                float4* mine = a.scratch + ((size_t)(cta * 2 + (cb >= ub ? 0 : 1)) * (2 * NT)) * kMegaConsumers + threadIdx.x;
#pragma unroll
                for (int j = 0; j < 2; ++j)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
                        mine[(size_t)(j * NT + nt) * kMegaConsumers] =
                            make_float4(acc[j][nt][0], acc[j][nt][1], acc[j][nt][2], acc[j][nt][3]);
                __threadfence();
                asm volatile("bar.sync 1, %0;" ::"n"(kMegaConsumers) : "memory");
                if (threadIdx.x == 0) {
                    // contributors: every CTA from i0 to i1 when each CTA owns at least one chunk; otherwise
                    // (fewer chunks than CTAs) every chunk of the unit belongs to a different CTA
                    const int n_contrib = T >= G ? i1 - i0 + 1 : CPR;
                    const int tk = atomicAdd(a.tickets + ph.ticket0 + u, 1);
                    *flag_s = (tk == n_contrib - 1) ? 1 : 0;
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kMegaConsumers) : "memory");
                const bool last = *flag_s != 0;   // rewritten only after the next named barrier
                if (threadIdx.x == 0) MEGA_TRACE(3);
                if (!last) continue;
                __threadfence();
#pragma unroll
                for (int j = 0; j < 2; ++j)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[j][nt][e] = 0.f;
                // contributions are fetched kBatch at a time (all loads of a batch in flight) and added in CTA order
                constexpr int kBatch = NT == 1 ? 8 : (NT == 2 ? 4 : 2);
                for (int ib = i0; ib <= i1; ib += kBatch) {
                    float4 v[kBatch][2 * NT];
#pragma unroll
                    for (int k = 0; k < kBatch; ++k) {
                        const int i = ib + k;
                        const bool on = i <= i1 && mega_begin(i, T, G) != mega_begin(i + 1, T, G);   // owns a chunk
                        const int slot = i * 2 + ((i == i0 && mega_begin(i0, T, G) < ub) ? 1 : 0);
                        const float4* src = a.scratch + ((size_t)slot * (2 * NT)) * kMegaConsumers + threadIdx.x;
#pragma unroll
                        for (int q = 0; q < 2 * NT; ++q)
                            v[k][q] = on ? __ldcg(src + (size_t)q * kMegaConsumers) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
#pragma unroll
                    for (int k = 0; k < kBatch; ++k)
#pragma unroll
                        for (int j = 0; j < 2; ++j)
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                acc[j][nt][0] += v[k][j * NT + nt].x;
                                acc[j][nt][1] += v[k][j * NT + nt].y;
                                acc[j][nt][2] += v[k][j * NT + nt].z;
                                acc[j][nt][3] += v[k][j * NT + nt].w;
                            }
                }
            }
            if (threadIdx.x == 0) MEGA_TRACE(4);
            if (mode == kPlain) mega_epilogue<NT, kPlain>(a, ph, u, warp, lane, acc, rstd_s, ssq_w);
            else if (mode == kQkvRope) mega_epilogue<NT, kQkvRope>(a, ph, u, warp, lane, acc, rstd_s, ssq_w);
            else if (mode == kResid) mega_epilogue<NT, kResid>(a, ph, u, warp, lane, acc, rstd_s, ssq_w);
            else mega_epilogue<NT, kSwiglu>(a, ph, u, warp, lane, acc, rstd_s, ssq_w);
            // publish: every thread's stores are ordered before the unit is counted as done (they will be read
            // by other SMs' bulk copies, i.e. through the asynchronous proxy, as well as by ordinary loads)
            fence_proxy_async_all();
            __threadfence();
            asm volatile("bar.sync 1, %0;" ::"n"(kMegaConsumers) : "memory");
            if (threadIdx.x == 0) MEGA_TRACE(5);
            if (threadIdx.x == 0) red_release_add(a.done + p, 1);
        }
    }
}

template <int NT>
static inline cudaError_t mega_launch_nt(const MegaArgs& a, int grid, cudaStream_t st) {
    return launch_pdl(mega_kernel<NT>, dim3(grid), dim3(kMegaThreads), (size_t)mega_smem_bytes(NT), st, a);
}
static inline cudaError_t mega_launch(int NT, const MegaArgs& a, int grid, cudaStream_t st) {
    switch (NT) {
        case 1: return mega_launch_nt<1>(a, grid, st);
        case 2: return mega_launch_nt<2>(a, grid, st);
        case 3: return mega_launch_nt<3>(a, grid, st);
        default: return mega_launch_nt<4>(a, grid, st);
    }
}
template <int NT>
static inline cudaError_t mega_set_attr() {
    cudaError_t e = cudaFuncSetAttribute(mega_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, mega_smem_bytes(NT));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(mega_kernel<NT>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
}
static inline cudaError_t mega_init_attrs() {
    cudaError_t e;
    if ((e = mega_set_attr<1>()) != cudaSuccess) return e;
    if ((e = mega_set_attr<2>()) != cudaSuccess) return e;
    if ((e = mega_set_attr<3>()) != cudaSuccess) return e;
    return mega_set_attr<4>();
}

// Host: geometry of one phase.
static inline void mega_phase_geometry(MegaPhase& ph, int N, int K) {
    ph.N = N;
    ph.KS = K / 16;
    ph.RB = (N + 127) / 128;
    ph.UB = (ph.RB + 1) / 2;
    ph.CPR = (ph.KS + kMegaKC - 1) / kMegaKC;
    ph.T = ph.UB * ph.CPR;
}

}  // namespace pipesd
