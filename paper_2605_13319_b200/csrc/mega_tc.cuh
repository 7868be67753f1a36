// Persistent layer-stack kernel for small token counts (M <= 32 rows) on the 5th-generation tensor cores.
//
// One CTA per SM stays resident for a whole sequence of GEMM "phases" (O projection, gate/up, down, the next
// layer's QKV, ..., LM head).  Every phase is cut into 256-row units x chunks of 4 k16-steps, and the flattened
// (unit, chunk) list is dealt out in equal contiguous ranges to the CTAs ("stream-K"), so that every SM streams
// the same number of weight bytes whatever the matrix shape.  Warp roles inside a CTA:
//   - weight producer (1 thread): walks the CTA's chunk list of ALL phases and keeps a 5-6 stage shared-memory
//     ring (32 KB of packed weights per stage) full with bulk asynchronous copies.  Weights depend on nothing,
//     so the stream runs ahead across phase boundaries; while the ring is full it pulls the chunks after the
//     ring's into L2, so that HBM keeps streaming while the SM waits at a boundary.
//   - activation producer (1 warp): waits until the phase that produces the input has finished everywhere (a
//     counter in global memory, released by the epilogues), then adds the matching activation chunk to each
//     stage and, where the phase normalises its input, derives the rows' RMSNorm factors.
//   - MMA issuer (1 thread): per chunk, eight tcgen05.mma (128 weight rows x 16 k  times  16 k x N token
//     columns, bf16 in, fp32 accumulators in tensor memory); the token columns are the split-bf16 hi terms
//     followed by the lo terms of the activations, so one instruction covers both.  tcgen05.commit hands a
//     stage back to the producers, and a finished accumulator (one of two) to the epilogue warps.
//   - eight epilogue warps: tcgen05.ld (thread = weight row, registers = tokens), hi + lo columns added, then
//     the fused epilogue (RoPE + K/V append | residual + next norm's gain and sum of squares | SwiGLU | plain).
// A unit whose chunks are spread over several CTAs is summed through global memory: contributors store their
// rows and count themselves in; the CTA that owns the unit's first chunk (for which the unit comes last in
// the phase) waits for the count and adds the contributions in CTA order -- a fixed order.  Every wait is
// bounded; a wait that gives up raises the device error word, which every other wait polls, so the kernel
// always terminates, and tensor memory is released on every path.
#pragma once
#include "common.cuh"
#include "gemm.cuh"

namespace pipesd {

constexpr int kMegaEpiWarps = 8;                           // warp w: 128-row block w >> 2, TMEM lane quarter w & 3
constexpr int kMegaEpiThreads = kMegaEpiWarps * 32;
constexpr int kMegaWarpW = 8, kMegaWarpX = 9, kMegaWarpMma = 10;
constexpr int kMegaThreads = 11 * 32;
constexpr int kMegaKC = 4;                                 // k16 steps per chunk
constexpr int kMegaWHalf = kMegaKC * 4096;                 // one 128-row block of a chunk
constexpr int kMegaWStage = 2 * kMegaWHalf;                // 256 rows
constexpr int kMegaMaxStages = 6;
constexpr int kMegaTail = 2048;                            // barriers | tmem base | rstd[32] | ssq exchange [8][32]
constexpr int kMegaMaxCtas = 160;
constexpr int kMegaSmemMax = 227 * 1024;
constexpr int kMegaTmemCols = 256;                         // 2 accumulators x 2 blocks x up to 64 columns
constexpr int kMegaL2Ahead = 8;                            // chunks a blocked weight producer pulls into L2
constexpr unsigned long long kMegaWaitNs = 1000000000ull;  // bound of every wait

__host__ __device__ constexpr int mega_stage_bytes(int NT) { return kMegaWStage + kMegaKC * NT * 512; }
__host__ __device__ constexpr int mega_stages(int NT) {
    return (kMegaSmemMax - kMegaTail) / mega_stage_bytes(NT) > kMegaMaxStages ? kMegaMaxStages
                                                                               : (kMegaSmemMax - kMegaTail) / mega_stage_bytes(NT);
}
__host__ __device__ constexpr int mega_smem_bytes(int NT) { return mega_stages(NT) * mega_stage_bytes(NT) + kMegaTail; }

// One GEMM of the chain.  Built once per context; lives in device memory.
struct MegaPhase {
    const uint4* W;        // weights in tensor-core operand order (see gemm_pack_umma_kernel)
    const uint4* xf;       // input activations of one token block, "xu" layout (see xu_piece_offset)
    int mode;              // GemmMode
    int N, KS, RB;         // logical rows, k16 steps, 128-row blocks
    int UB, CPR, T;        // 256-row units, chunks per unit, chunks in the phase
    int ticket0;           // first contribution counter of the phase
    const float* ssq_in;   // sums of squares of the un-normalised input rows [n_ssq][M] (null: no input norm)
    int n_ssq;
    int layer;             // kQkvRope
    float* out;            // kPlain [M][N]
    float* x;              // kResid: residual stream [M][N]
    uint16_t* xf_out;      // kResid: x_new * gain_next in xu layout;  kSwiglu: silu(gate)*up in xu layout
    const float* gain_next;
    float* ssq_out;        // kResid: [UB][M]
};

struct MegaArgs {
    const MegaPhase* phases;
    int p0, p1;            // phase range of this launch
    int launch_idx;        // position of this launch in the pass
    int M;
    int* done;             // [n_phases] finished units per phase (zero at the start of a pass)
    int* tickets;          // per (phase, unit) contribution counters (zero at the start of a pass)
    int* arrived;          // CTAs of this launch that have started
    float4* scratch;       // rows of a CTA's part of a shared unit: [cta][2*NT][256]
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

// ---- weights in tensor-core operand order -----------------------------------------------------------------
// Per (128-row block rb, k16 step ks) 4 KB: the K-major, unswizzled operand layout of tcgen05.mma -- 8x8
// "core matrices" (8 rows x 16 bytes, contiguous), the two k halves of a row group 128 bytes apart, row groups
// 256 bytes apart.  Packed rows map to logical rows per `mode` exactly as in gemm_pack_kernel (a rotary pair /
// a gate-up pair sits in rows i and i + 8 of a 16-row tile); rows beyond the sources are zero.
__global__ void gemm_pack_umma_kernel(PackSrc src, uint4* __restrict__ packed, int n_rows, int K) {
    const int KS = K / 16;
    const int n_rb = (n_rows + 127) / 128;
    const size_t total = (size_t)n_rb * 128 * KS * 2;        // 16-byte pieces
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int kgq = (int)(i % (2 * KS));                 // k8 group along the row
        const int pr = (int)(i / (2 * KS));                  // packed row
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (pr < n_rows) {
            int lr, which = 0;
            if (src.mode == kSwiglu) { which = (pr & 15) < 8 ? 0 : 1; lr = gu_feature(pr); }
            else {
                lr = src.mode == kQkvRope ? qkv_logical_row(pr, src.hd) : pr;
                while (which < 2 && lr >= src.rows[which]) { lr -= src.rows[which]; ++which; }
            }
            v = *reinterpret_cast<const uint4*>(src.w[which] + (size_t)lr * K + 8 * kgq);
        }
        const int rb = pr >> 7, r = pr & 127, ks = kgq >> 1, kg = kgq & 1;
        packed[((size_t)rb * KS + ks) * 256 + ((r >> 3) * 2 + kg) * 8 + (r & 7)] = v;
    }
}

// ---- tcgen05 wrappers ------------------------------------------------------------------------------------
// Shared-memory matrix descriptor, no swizzle: start address, leading (K-direction for a K-major operand, see
// the operand comments) and stride byte offsets between core matrices, all in 16-byte units.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46);
}
// Instruction descriptor: fp32 accumulate, bf16 A (K-major) and B (token-major), M = 128, N columns.
__host__ __device__ constexpr uint32_t umma_idesc(int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((uint32_t)(N >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t"
        "}\n"
        :
        : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// The barrier receives one arrival when every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 8 consecutive fp32 columns of this thread's TMEM lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&r)[8]) {
    uint32_t u[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7])
                 : "r"(taddr));
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = __uint_as_float(u[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

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

__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// mbarrier wait that also gives up when another part of the grid has raised the error word.
__device__ __forceinline__ bool mbar_wait_err(uint32_t bar, uint32_t parity, const int* err) {
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try(bar, parity)) return true;
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
__device__ __forceinline__ int mega_owner(int c, int T, int G) { return (int)((((unsigned)c + 1u) * (unsigned)G - 1u) / (unsigned)T); }
__device__ __forceinline__ int mega_begin(int i, int T, int G) { return (int)(((unsigned)T * (unsigned)i) / (unsigned)G); }

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

// 8 fp32 values -> 8 bf16 hi terms and 8 bf16 lo terms, each one 16-byte word.
__device__ __forceinline__ void split8(const float* v, uint4& hi, uint4& lo) {
    uint16_t h[8], l[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) split_bf16(v[i], h[i], l[i]);
    hi = make_uint4(pack2(h[0], h[1]), pack2(h[2], h[3]), pack2(h[4], h[5]), pack2(h[6], h[7]));
    lo = make_uint4(pack2(l[0], l[1]), pack2(l[2], l[3]), pack2(l[4], l[5]), pack2(l[6], l[7]));
}

// Per-token sums over the 32 lanes of a warp by recursive halving (MTP values per lane in, MTP a power of two):
// after the exchange steps every lane holds the sum of ONE token over the lanes that differ from it in the
// exchanged bits; the remaining bits are folded by plain butterfly adds.  Returns the sum, `tok` says whose.
template <int MTP>
__device__ __forceinline__ float warp_token_sums(float (&s)[MTP], int lane, int& tok) {
    tok = 0;
    int mask = 16;
#pragma unroll
    for (int h = MTP / 2; h >= 1; h >>= 1) {
        const bool up = (lane & mask) != 0;
#pragma unroll
        for (int i = 0; i < h; ++i) {
            const float keep = up ? s[i + h] : s[i], send = up ? s[i] : s[i + h];
            s[i] = keep + __shfl_xor_sync(0xffffffffu, send, mask);
        }
        if (up) tok += h;
        mask >>= 1;
    }
    float r = s[0];
    for (; mask >= 1; mask >>= 1) r += __shfl_xor_sync(0xffffffffu, r, mask);
    return r;
}

// Epilogue of one finished 256-row unit.  Thread (warp, lane) owns packed row u*256 + warp*32 + lane and holds
// its value for every token.  The fused layouts put a rotary pair / a (gate, up) pair in rows i and i + 8 of a
// 16-row tile: lanes l and l ^ 8.
template <int NT, int MODE>
__device__ __forceinline__ void mega_epilogue(const MegaArgs& a, const MegaPhase& ph, int u, int warp, int lane,
                                              float (&v)[NT * 8], const float* rstd_s, float* ssq_w) {
    constexpr int MT = NT * 8;
    const int N = ph.N, M = a.M;
    const int pr = u * 256 + warp * 32 + lane;
    const bool row_live = pr < N;
    if (ph.ssq_in != nullptr) {
#pragma unroll
        for (int t = 0; t < MT; ++t) v[t] *= rstd_s[t];
    }
    if (MODE == kPlain) {
        if (row_live) {
#pragma unroll
            for (int t = 0; t < MT; ++t)
                if (t < M) ph.out[(size_t)t * N + pr] = v[t];
        }
        return;
    }
    if (MODE == kResid) {
        constexpr int MTP = MT <= 8 ? 8 : (MT <= 16 ? 16 : 32);
        float xv[MT], sq[MTP];
#pragma unroll
        for (int t = 0; t < MT; ++t) xv[t] = (row_live && t < M) ? __ldcg(ph.x + (size_t)t * N + pr) : 0.f;
        const float gain = row_live ? ph.gain_next[pr] : 0.f;
#pragma unroll
        for (int t = 0; t < MTP; ++t) sq[t] = 0.f;
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            const float xn = xv[t] + v[t];
            if (row_live && t < M) {
                ph.x[(size_t)t * N + pr] = xn;
                sq[t] = xn * xn;
            }
            v[t] = (t < M) ? xn * gain : 0.f;
        }
        if (row_live) {
            // this row is k index pr of the next projection: one 16-byte piece per 8 tokens, hi and lo
            unsigned char* dst = reinterpret_cast<unsigned char*>(ph.xf_out) + xu_piece_offset(pr, 0, NT);
#pragma unroll
            for (int ng = 0; ng < NT; ++ng) {
                uint4 hi, lo;
                split8(&v[8 * ng], hi, lo);
                *reinterpret_cast<uint4*>(dst + ng * 128) = hi;
                *reinterpret_cast<uint4*>(dst + (NT + ng) * 128) = lo;
            }
        }
        // sums of squares of the unit's 256 rows per token: inside a warp by recursive halving, over the 8
        // warps through shared memory, both in a fixed order
        int tok;
        const float r = warp_token_sums<MTP>(sq, lane, tok);
        constexpr int kRest = 32 / MTP - 1;                    // lane bits not consumed by the exchange steps
        if ((lane & kRest) == 0) ssq_w[warp * 32 + tok] = r;
        asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
        const int t = threadIdx.x;
        if (t < MT && t < M) {
            float q = 0.f;
#pragma unroll
            for (int w = 0; w < kMegaEpiWarps; ++w) q += ssq_w[w * 32 + t];
            ph.ssq_out[(size_t)u * M + t] = q;
        }
        return;
    }
    const bool upper = (lane & 8) != 0;
    if (MODE == kSwiglu) {
        // lanes l (gate) and l ^ 8 (up) hold feature (pr >> 4) * 8 + (l & 7); both compute the product, the gate
        // lane stores the hi pieces and the up lane the lo pieces
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            const float other = __shfl_xor_sync(0xffffffffu, v[t], 8);
            const float gt = upper ? other : v[t], up = upper ? v[t] : other;
            v[t] = (t < M) ? gt / (1.f + expf(-gt)) * up : 0.f;
        }
        if ((pr | 8) < N) {
            const int f = (pr >> 4) * 8 + (lane & 7);
            unsigned char* dst = reinterpret_cast<unsigned char*>(ph.xf_out) + xu_piece_offset(f, upper ? NT : 0, NT);
#pragma unroll
            for (int ng = 0; ng < NT; ++ng) {
                uint4 hi, lo;
                split8(&v[8 * ng], hi, lo);
                *reinterpret_cast<uint4*>(dst + ng * 128) = upper ? lo : hi;
            }
        }
        return;
    }
    // kQkvRope: lanes l and l ^ 8 hold dims dim and dim + hd/2 of one head
    {
        const int hd = a.hd, half = hd / 2;
        const int head = pr / hd, within = pr - head * hd;
        const int dlow = 8 * (within >> 4) + (lane & 7);          // dim of the pair's first element
        const int dim = upper ? dlow + half : dlow;
        const bool rot = head < a.Hq + a.Hkv;
        const int kv = head < a.Hq + a.Hkv ? 0 : 1;
        const int kvh = kv ? head - a.Hq - a.Hkv : head - a.Hq;
        const size_t per_head = (size_t)a.page_size * hd;
        const size_t kv_base = (size_t)ph.layer * a.n_pages * 2 * a.Hkv * per_head + ((size_t)kv * a.Hkv + kvh) * per_head + dim;
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            const float other = __shfl_xor_sync(0xffffffffu, v[t], 8);
            float o = v[t];
            if (rot && row_live && t < M) {
                const float c = a.cs[(size_t)t * half + dlow], s = a.sn[(size_t)t * half + dlow];
                o = upper ? v[t] * c + other * s : v[t] * c - other * s;
            }
            // K/V: neighbouring dims of one token travel as one 4-byte store
            const uint32_t mine = f32_to_bf16_bits(o);
            const uint32_t nb = __shfl_xor_sync(0xffffffffu, mine, 1);
            if (row_live && t < M) {
                if (head < a.Hq) a.q_out[((size_t)t * a.Hq + head) * hd + dim] = o;
                else if ((lane & 1) == 0)
                    *reinterpret_cast<uint32_t*>(a.kv_pool + (size_t)a.row_kvoff[t] + kv_base) = mine | (nb << 16);
            }
        }
    }
}

template <int NT>
__global__ void __launch_bounds__(kMegaThreads, 1) mega_kernel(const MegaArgs a) {
    constexpr int kStage = mega_stage_bytes(NT);
    constexpr int kStages = mega_stages(NT);
    constexpr int MT = NT * 8;
    constexpr int kCols = 2 * MT;                 // token columns of one accumulator block: hi terms | lo terms
    constexpr int kAccCols = 2 * kCols;           // one accumulator = two 128-row blocks
    static_assert(2 * kAccCols <= kMegaTmemCols, "tensor memory budget");
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* tail = smem + kStages * kStage;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);          // fullW[8] | fullX[8] | empty[8] | accfull[2] | accempty[2] | drain | rstd
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 256);
    float* rstd_s = reinterpret_cast<float*>(tail + 384);        // [32]
    float* ssq_w = reinterpret_cast<float*>(tail + 512);         // [8][32]
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t fullW0 = smem_u32(bars), fullX0 = fullW0 + 64, empty0 = fullW0 + 128;
    const uint32_t accfull0 = fullW0 + 192, accempty0 = fullW0 + 208, drain0 = fullW0 + 224, rstd0 = fullW0 + 232;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = (int)gridDim.x, cta = (int)blockIdx.x;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(fullW0 + 8 * i, 1);
            mbar_init(fullX0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(accfull0 + 8 * i, 1);
            mbar_init(accempty0 + 8 * i, kMegaEpiWarps);
        }
        mbar_init(drain0, 1);
        mbar_init(rstd0, 1);
        fence_mbar_init();
        red_release_add(a.arrived, 1);
    }
    if (warp == kMegaWarpMma) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)kMegaTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == kMegaWarpW) {
        // ------------------------------------------------ weight producer: runs ahead of everything
        if (lane == 0) {
            MegaWalk ring, pf;               // next chunk for the ring / next chunk to prefetch into L2
            ring.start(a, cta, G);
            pf = ring;
            int n = 0, st = 0, n_pf = 0;
            bool ok = true;
            while (ring.valid()) {
                if (n >= kStages) {
                    // Ring full: the MMAs are held up (usually at a phase boundary).  HBM must not go idle
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
        }
    } else if (warp == kMegaWarpX) {
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
            } else {
                // lanes 1..31: the input rows' RMSNorm factors, needed only by the epilogue, computed while
                // lane 0's copies are in flight and handed to the epilogue warps through their own barrier
                if (ph.ssq_in != nullptr) {
                    for (int t = lane - 1; t < MT; t += 31) {
                        float part[32], ss = 0.f;    // d_model <= 8192: at most 32 units; all loads in flight together
#pragma unroll
                        for (int b = 0; b < 32; ++b)
                            part[b] = (t < a.M && b < ph.n_ssq) ? __ldcg(ph.ssq_in + (size_t)b * a.M + t) : 0.f;
#pragma unroll
                        for (int b = 0; b < 32; ++b) ss += part[b];
                        rstd_s[t] = rsqrtf(ss / (float)a.d_in + a.eps);
                    }
                    __syncwarp(0xfffffffeu);
                    if (lane == 1) mbar_arrive(rstd0);
                }
            }
            __syncwarp();
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
    } else if (warp == kMegaWarpMma) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc(kCols);
            int n = 0, st = 0, seg = 0;
            bool ok = true;
            for (int p = a.p0; p < a.p1; ++p) {
                const MegaPhase& ph = a.phases[p];
                const int T = ph.T, CPR = ph.CPR, KS = ph.KS, RB = ph.RB;
                const int cb = mega_begin(cta, T, G), ce = mega_begin(cta + 1, T, G);
                int c = cb;
                while (c < ce) {
                    const int u = c / CPR, ub = u * CPR;
                    const int se = ce < ub + CPR ? ce : ub + CPR;
                    const bool two = 2 * u + 1 < RB;
                    const int buf = seg & 1;
                    // the accumulator is free once the epilogue warps have read its previous contents
                    if (ok && seg >= 2) ok = mbar_wait_err(accempty0 + 8 * buf, (uint32_t)((seg >> 1) - 1) & 1u, a.err);
                    tc_fence_after();
                    const uint32_t d0 = tmem + (uint32_t)(buf * kAccCols);
                    uint32_t accumulate = 0;
                    for (; c < se; ++c, ++n) {
                        if (ok) {
                            const uint32_t par = (uint32_t)(n / kStages) & 1u;
                            ok = mbar_wait_err(fullW0 + 8 * st, par, a.err) && mbar_wait_err(fullX0 + 8 * st, par, a.err);
                            if (!ok) atomicCAS(a.err, 0, 13);
                        }
                        if (ok) {
                            tc_fence_after();
                            const int ks = (c - ub) * kMegaKC;
                            const int kc = KS - ks < kMegaKC ? KS - ks : kMegaKC;
                            const uint32_t wst = smem_base + st * kStage, xst = wst + kMegaWStage;
                            for (int k = 0; k < kc; ++k) {
                                // A: 128 rows x 16 k, K-major: k halves 128 B apart (leading), row groups 256 B (stride)
                                // B: 16 k x kCols tokens, token-major: k halves NT*256 B apart (leading), token groups 128 B
                                const uint64_t bdesc = umma_desc(xst + k * NT * 512, NT * 256, 128);
                                umma_bf16(d0, umma_desc(wst + k * 4096, 128, 256), bdesc, idesc, accumulate);
                                if (two) umma_bf16(d0 + kCols, umma_desc(wst + kMegaWHalf + k * 4096, 128, 256), bdesc, idesc, accumulate);
                                accumulate = 1;
                            }
                            umma_commit(empty0 + 8 * st);      // the stage is free when these MMAs have read it
                        }
                        if (++st == kStages) st = 0;
                    }
                    if (ok) umma_commit(accfull0 + 8 * buf);
                    ++seg;
                }
            }
            // every MMA issued has completed before tensor memory is released
            umma_commit(drain0);
            mbar_wait(drain0, 0);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue warps
        pdl_wait();      // epilogues read what earlier kernels wrote (rotary tables, K/V offsets, residual stream)
        int seg = 0, n_norm = 0;      // n_norm: phases so far whose input is normalised and in which this CTA has work
        bool ok = true;
        const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * kCols);
        for (int p = a.p0; p < a.p1; ++p) {
            const MegaPhase& ph = a.phases[p];
            const int T = ph.T, CPR = ph.CPR, mode = ph.mode;
            const int cb = mega_begin(cta, T, G), ce = mega_begin(cta + 1, T, G);
            int c = cb;
            if (cb < ce && ph.ssq_in != nullptr) {
                // the activation producer has derived this phase's RMSNorm factors
                if (ok) {
                    ok = mbar_wait_err(rstd0, (uint32_t)n_norm & 1u, a.err);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok && lane == 0) atomicCAS(a.err, 0, 16);
                }
                ++n_norm;
            }
            while (c < ce) {
                const int u = c / CPR, ub = u * CPR;
                const int se = ce < ub + CPR ? ce : ub + CPR;
                c = se;
                const int buf = seg & 1;
                // A wait that gave up is not an exit: the warp keeps walking the schedule (without waiting) so
                // that it still meets the other epilogue warps at every named barrier below.
                if (ok) {
                    ok = mbar_wait_err(accfull0 + 8 * buf, (uint32_t)(seg >> 1) & 1u, a.err);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok && lane == 0) atomicCAS(a.err, 0, 15);
                }
                float v[MT];
                if (ok) {
                    tc_fence_after();
                    float hi[NT][8], lo[NT][8];
#pragma unroll
                    for (int ng = 0; ng < NT; ++ng) {
                        tmem_ld8(t_lane + buf * kAccCols + ng * 8, hi[ng]);
                        tmem_ld8(t_lane + buf * kAccCols + MT + ng * 8, lo[ng]);
                    }
                    tmem_ld_wait();
#pragma unroll
                    for (int ng = 0; ng < NT; ++ng)
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[ng * 8 + i] = hi[ng][i] + lo[ng][i];
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(accempty0 + 8 * buf);
                } else {
#pragma unroll
                    for (int t = 0; t < MT; ++t) v[t] = 0.f;
                }
                ++seg;
                if (threadIdx.x == 0) MEGA_TRACE(2);
                // ---- the CTA's part of unit u is summed.  Alone on the unit: epilogue.  Otherwise the CTA that
                // owns the unit's first chunk collects (the unit is the last thing that CTA does in the phase,
                // so it waits for little): the others leave their rows in global memory and count themselves
                // in; the collector waits for that count, adds the contributions to its own in CTA order (a
                // fixed order), and runs the epilogue.  Contributors never wait.
                const int i0 = mega_owner(ub, T, G), i1 = mega_owner(ub + CPR - 1, T, G);
                if (i0 != i1) {
                    if (cta != i0) {
                        float4* mine = a.scratch + ((size_t)cta * (2 * NT)) * kMegaEpiThreads + threadIdx.x;
#pragma unroll
                        for (int q = 0; q < 2 * NT; ++q)
                            mine[(size_t)q * kMegaEpiThreads] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                        // all stores of the CTA happen before thread 0's release (ordered by the named barrier)
                        asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
                        if (threadIdx.x == 0) red_release_add(a.tickets + ph.ticket0 + u, 1);
                        if (threadIdx.x == 0) MEGA_TRACE(3);
                        continue;
                    }
                    if (threadIdx.x == 0) {
                        // contributors: every CTA from i0 to i1 when each CTA owns at least one chunk; otherwise
                        // (fewer chunks than CTAs) every chunk of the unit belongs to a different CTA
                        const int n_contrib = T >= G ? i1 - i0 + 1 : CPR;
                        if (!poll_counter(a.tickets + ph.ticket0 + u, n_contrib - 1, a.err)) atomicCAS(a.err, 0, 14);
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
                    if (threadIdx.x == 0) MEGA_TRACE(3);
                    // contributions are fetched kBatch at a time (all loads of a batch in flight)
                    constexpr int kBatch = NT == 1 ? 8 : (NT == 2 ? 4 : 2);
                    for (int ib = i0 + 1; ib <= i1; ib += kBatch) {
                        float4 w[kBatch][2 * NT];
#pragma unroll
                        for (int k = 0; k < kBatch; ++k) {
                            const int i = ib + k;
                            const bool on = i <= i1 && (T >= G || mega_begin(i, T, G) != mega_begin(i + 1, T, G));
                            const float4* src = a.scratch + ((size_t)i * (2 * NT)) * kMegaEpiThreads + threadIdx.x;
#pragma unroll
                            for (int q = 0; q < 2 * NT; ++q)
                                w[k][q] = on ? __ldcg(src + (size_t)q * kMegaEpiThreads) : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int k = 0; k < kBatch; ++k)
#pragma unroll
                            for (int q = 0; q < 2 * NT; ++q) {
                                v[4 * q] += w[k][q].x;
                                v[4 * q + 1] += w[k][q].y;
                                v[4 * q + 2] += w[k][q].z;
                                v[4 * q + 3] += w[k][q].w;
                            }
                    }
                }
                if (threadIdx.x == 0) MEGA_TRACE(4);
                if (mode == kPlain) mega_epilogue<NT, kPlain>(a, ph, u, warp, lane, v, rstd_s, ssq_w);
                else if (mode == kQkvRope) mega_epilogue<NT, kQkvRope>(a, ph, u, warp, lane, v, rstd_s, ssq_w);
                else if (mode == kResid) mega_epilogue<NT, kResid>(a, ph, u, warp, lane, v, rstd_s, ssq_w);
                else mega_epilogue<NT, kSwiglu>(a, ph, u, warp, lane, v, rstd_s, ssq_w);
                // publish: the named barrier orders every thread's stores before thread 0's release; readers
                // acquire the counter (and fence the asynchronous proxy before their bulk copies)
                asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
                if (threadIdx.x == 0) MEGA_TRACE(5);
                if (threadIdx.x == 0) red_release_add(a.done + p, 1);
            }
        }
    }
    // ---- every role ends here: tensor memory goes back before the CTA exits, on every path
    tc_fence_before();
    __syncthreads();
    if (warp == kMegaWarpMma) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kMegaTmemCols) : "memory");
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
