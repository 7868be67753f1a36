// Persistent layer-stack kernel for small token counts (M <= 32 rows) on the 5th-generation tensor cores.
//
// One CTA per SM stays resident for a whole sequence of GEMM "phases" (O projection, gate/up, down, the next
// layer's QKV, ..., LM head).  Every phase is cut into 256-row units x chunks of 4 k16-steps, and the flattened
// (unit, chunk) list is dealt out in equal contiguous ranges to the CTAs ("stream-K"), so that every SM streams
// the same number of weight bytes whatever the matrix shape.  Warp roles inside a CTA:
//   - weight producer (1 thread): walks the CTA's chunk list of ALL phases and keeps a 5-6 stage shared-memory
//     ring (32 KB of packed weights per stage) full with bulk asynchronous copies, at most three outstanding
//     (more only queues in front of the boundaries' small latency-critical accesses).  Weights depend on
//     nothing, so the stream runs ahead across phase boundaries.  The copies carry an L2 evict-first hint.
//   - activation producer (1 warp): waits until the phase that produces the input has finished everywhere (a
//     counter in global memory, released by the epilogues), then adds the matching activation chunk to each
//     stage and, where the phase normalises its input, derives the rows' RMSNorm factors.
//   - MMA issuer (1 thread): per chunk, eight tcgen05.mma (128 weight rows x 16 k  times  16 k x N token
//     columns, bf16 in, fp32 accumulators in tensor memory); the token columns are the split-bf16 hi terms
//     followed by the lo terms of the activations, so one instruction covers both.  tcgen05.commit hands a
//     stage back to the producers, and a finished accumulator (one of two) to the epilogue warps.
//   - eight epilogue warps: tcgen05.ld (thread = weight row, registers = tokens), hi + lo columns added, then
//     the fused epilogue (RoPE + K/V append | residual + next norm's gain and sum of squares | SwiGLU | plain).
//   - publisher (1 thread): tells the other CTAs that a segment of this CTA is finished (a release on a global
//     counter, i.e. a fence over the CTA's stores), so that no epilogue warp spends that microsecond.
// A unit whose chunks are spread over several CTAs is summed through global memory: contributors store their
// rows and count themselves in; the CTA that owns the unit's first chunk (for which the unit comes last in
// the phase) waits for the count and adds the contributions in CTA order -- a fixed order.
// An attention phase (single-request passes) runs in the same ring: its chunks are 64-key tiles of one KV head
// (K rows + V rows = one stage, fetched page by page), consumed by the eight epilogue warps (att_segment).
// Every wait is bounded; a wait that gives up raises the device error word, which every other wait polls, so the
// kernel always terminates, and tensor memory is released on every path.
#pragma once
#include "common.cuh"
#include "gemm.cuh"

namespace pipesd {

constexpr int kMegaEpiWarps = 8;                           // warp w: 128-row block w >> 2, TMEM lane quarter w & 3
constexpr int kMegaEpiThreads = kMegaEpiWarps * 32;
constexpr int kMegaWarpW = 8, kMegaWarpX = 9, kMegaWarpMma = 10, kMegaWarpPub = 11;
constexpr int kMegaThreads = 12 * 32;
constexpr int kMegaKC = 4;                                 // k16 steps per chunk
constexpr int kMegaWHalf = kMegaKC * 4096;                 // one 128-row block of a chunk
constexpr int kMegaWStage = 2 * kMegaWHalf;                // 256 rows
constexpr int kMegaMaxStages = 6;
constexpr int kMegaTail = 2048;                            // barriers | tmem base | rstd[32] | ssq exchange [8][32]
constexpr int kMegaQArea = 8192;                           // attention phases: the head's queries as MMA A fragments (hi | lo)
constexpr int kPhaseAttn = 4;                              // MegaPhase::mode of an attention phase (the GEMM modes are 0..3)
constexpr int kAttTile = 64;                               // keys per attention chunk: K tile + V tile fill a ring stage
constexpr int kMegaMaxCtas = 160;
constexpr int kMegaSmemMax = 227 * 1024;
constexpr int kMegaTmemCols = 256;                         // 2 accumulators x 2 blocks x up to 64 columns
constexpr int kMegaMaxInFlight = 3;                        // weight chunks one CTA has outstanding at a time (see the weight producer)
constexpr unsigned long long kMegaWaitNs = 1000000000ull;  // bound of every wait

__host__ __device__ constexpr int mega_stage_bytes(int NT) { return kMegaWStage + kMegaKC * NT * 512; }
__host__ __device__ constexpr int mega_stages(int NT) {
    return (kMegaSmemMax - kMegaTail - kMegaQArea) / mega_stage_bytes(NT) > kMegaMaxStages
               ? kMegaMaxStages
               : (kMegaSmemMax - kMegaTail - kMegaQArea) / mega_stage_bytes(NT);
}
__host__ __device__ constexpr int mega_smem_bytes(int NT) { return mega_stages(NT) * mega_stage_bytes(NT) + kMegaTail + kMegaQArea; }

// One GEMM of the chain, or one attention phase (mode == kPhaseAttn: UB = KV heads, layer and xf_out set; the
// number of key tiles per head changes from pass to pass and comes with the launch arguments).  Built once per
// context; lives in device memory.
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
    // attention phases (one request per pass): keys [0, att_base) are cached, [att_base, att_base + att_rows) are
    // this pass's rows; att_cpr = tiles of 64 keys per head
    int att_base, att_rows, att_cpr;
    const int32_t* att_bt;   // the request's block table row
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
__device__ __forceinline__ void st_release_cta(int* smem_p, int v) {
    asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(smem_p)), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_cta(const int* smem_p) {
    int v;
    asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(smem_p)) : "memory");
    return v;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }


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

__device__ __forceinline__ int phase_cpr(const MegaArgs& a, const MegaPhase& ph) { return ph.mode == kPhaseAttn ? a.att_cpr : ph.CPR; }
__device__ __forceinline__ int phase_chunks(const MegaArgs& a, const MegaPhase& ph) {
    return ph.mode == kPhaseAttn ? a.att_cpr * ph.UB : ph.T;
}

// Cursor over one CTA's chunks (weights, or K/V tiles of an attention phase) through the phases of a launch.
struct MegaWalk {
    int p, p1, c, ce, u, cc, KS, CPR, RB, mode, layer;
    const unsigned char* W;
    __device__ __forceinline__ void load_phase(const MegaArgs& a, int cta, int G) {
        for (; p < p1; ++p) {
            const MegaPhase& ph = a.phases[p];
            const int T = phase_chunks(a, ph);
            c = mega_begin(cta, T, G);
            ce = mega_begin(cta + 1, T, G);
            if (c < ce) {
                KS = ph.KS; CPR = phase_cpr(a, ph); RB = ph.RB; mode = ph.mode; layer = ph.layer;
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
};

// Attention chunk (KV head `kvh`, key tile `tile`): copies the pages of the tile into a stage -- K rows at the
// stage's start, V rows 64 rows further -- and returns the bytes to expect.  `fresh` selects which pages: false
// = pages made only of keys cached before this pass (they depend on nothing: the weight producer's share), true
// = pages that hold rows of this pass (the activation producer's share, after the QKV phase has finished).
// Pages hold 16 positions (the host admits nothing else to these phases).
__device__ __forceinline__ uint32_t att_issue_pages(const MegaArgs& a, int layer, int kvh, int tile, bool fresh, int4 pages,
                                                    uint32_t stage_addr, uint32_t bar, bool dry) {
    const int total = a.att_base + a.att_rows;
    const uint32_t blk = 16u * (uint32_t)a.hd * 2u;                 // one page of one head: K or V
    const int pg[4] = {pages.x, pages.y, pages.z, pages.w};
    uint32_t bytes = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int pos0 = tile * kAttTile + 16 * q;
        if (pos0 >= total) continue;
        const bool is_fresh = pos0 + 16 > a.att_base;
        if (is_fresh != fresh) continue;
        bytes += 2 * blk;
        if (dry) continue;
        const uint16_t* k = a.kv_pool + kv_index(layer, a.n_pages, pg[q], 0, a.Hkv, kvh, 16, 0, a.hd, 0);
        bulk_g2s(stage_addr + q * blk, k, blk, bar);
        bulk_g2s(stage_addr + 4 * blk + q * blk, k + (size_t)a.Hkv * 16 * a.hd, blk, bar);
    }
    return bytes;
}
__device__ __forceinline__ int4 att_tile_pages(const MegaArgs& a, int tile) {
    return __ldcg(reinterpret_cast<const int4*>(a.att_bt) + tile);      // 4 pages of 16 positions per 64-key tile
}

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
__device__ __forceinline__ void mega_epilogue(const MegaArgs& a, const MegaPhase& ph, int p, int cta, int u, int warp, int lane,
                                              float (&v)[NT * 8], const float (&pa)[NT * 8], const float (&pb)[NT * 8],
                                              const float* rstd_s, float* ssq_w, const long long* kvoff_s) {
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
        float sq[MTP];
        const float gain = pb[0];                    // pa: the row's residual values, fetched when the unit started
#pragma unroll
        for (int t = 0; t < MTP; ++t) sq[t] = 0.f;
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            if (t < M) {                              // uniform: rows of padding tokens cost nothing
                const float xn = pa[t] + v[t];
                if (row_live) {
                    ph.x[(size_t)t * N + pr] = xn;
                    sq[t] = xn * xn;
                }
                v[t] = xn * gain;
            } else {
                v[t] = 0.f;
            }
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
            if (t < M) {                              // uniform
                const float other = __shfl_xor_sync(0xffffffffu, v[t], 8);
                const float gt = upper ? other : v[t], up = upper ? v[t] : other;
                v[t] = gt / (1.f + expf(-gt)) * up;
            } else {
                v[t] = 0.f;
            }
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
        const size_t kv_base = (size_t)ph.layer * a.n_pages * 2 * a.Hkv * per_head + ((size_t)kv * a.Hkv + kvh) * per_head;
        // pa / pb: the rotary factors of this row's dim for every token, fetched when the unit started
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            if (t >= M) break;                        // uniform
            const float other = __shfl_xor_sync(0xffffffffu, v[t], 8);
            const float o = rot ? (upper ? v[t] * pa[t] + other * pb[t] : v[t] * pa[t] - other * pb[t]) : v[t];
            // K/V: neighbouring dims of one token travel as one 4-byte store
            const uint32_t mine = f32_to_bf16_bits(o);
            const uint32_t nb = __shfl_xor_sync(0xffffffffu, mine, 1);
            if (row_live) {
                if (head < a.Hq) a.q_out[((size_t)t * a.Hq + head) * hd + dim] = o;
                else if ((lane & 1) == 0) {
                    const long long ko = kvoff_s[t];
                    *reinterpret_cast<uint32_t*>(a.kv_pool + (size_t)(ko & ~7ll) + kv_base + kv_swizzle(dim, (int)(ko & 7))) =
                        mine | (nb << 16);
                }
            }
        }
    }
}

// What the epilogue of unit u will read from global memory besides the accumulators, fetched before the
// accumulators are waited for (none of it depends on the phase in progress): kResid -- the row's residual values
// (pa) and the next norm's gain (pb[0]); kQkvRope -- cos (pa) and sin (pb) of the row's dim for every token.
template <int NT>
__device__ __forceinline__ void mega_preload(const MegaArgs& a, const MegaPhase& ph, int u, int warp, int lane,
                                             float (&pa)[NT * 8], float (&pb)[NT * 8]) {
    constexpr int MT = NT * 8;
    const int N = ph.N, M = a.M;
    const int pr = u * 256 + warp * 32 + lane;
    const bool row_live = pr < N;
    if (ph.mode == kResid) {
#pragma unroll
        for (int t = 0; t < MT; ++t) pa[t] = (row_live && t < M) ? __ldcg(ph.x + (size_t)t * N + pr) : 0.f;
        pb[0] = row_live ? ph.gain_next[pr] : 0.f;
    } else if (ph.mode == kQkvRope) {
        const int hd = a.hd, half = hd / 2;
        const int head = pr / hd, within = pr - head * hd;
        const int dlow = 8 * (within >> 4) + (lane & 7);
        const bool rot = row_live && head < a.Hq + a.Hkv;
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            pa[t] = (rot && t < M) ? a.cs[(size_t)t * half + dlow] : 1.f;
            pb[t] = (rot && t < M) ? a.sn[(size_t)t * half + dlow] : 0.f;
        }
    }
}

// ---- attention phase: one segment = one KV head x a run of 64-key tiles, consumed by the eight epilogue warps --
__device__ __forceinline__ void mma_bf16_1688(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ float ex2_approx(float x) {   // 2^x, relative error 2^-22; 2^-inf = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void split2(float a, float b, uint32_t& hi, uint32_t& lo) {   // packed bf16x2 hi and lo terms
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    const float2 hf = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(a - hf.x, b - hf.y);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

// The (at most 16) query rows that share KV head `kvh` -- every (query head of the group, chunk row) pair --
// attend to the keys of tiles [tile0, tile1).  A tile is 64 keys: K rows at the start of a ring stage, V rows
// behind them, rows chunk-permuted as in the pool.  Warp w takes keys 8w..8w+7 of every tile: Q K^T on
// m16n8k16 (Q split into bf16 hi + lo), online softmax in the log2 domain, P V on m16n8k8 (P split likewise).
// At the end the eight warps' running (max, sum, output) are merged through the last stage's shared memory in a
// fixed order; heads whose tiles are spread over several CTAs are merged through global memory by the CTA that
// owns the head's first tile, exactly as the GEMM units are, and the normalised output goes to the output
// projection's input array.  Every named barrier below is reached by all 256 threads, also after a failed wait.
template <int HD>
__device__ __forceinline__ void att_segment(const MegaArgs& a, const MegaPhase& ph, int p, int cta, int G, int kvh, int tile0, int tile1,
                                            int ub, int T, int CPR, int NT, int kStages, int kStage, unsigned char* smem,
                                            uint32_t fullW0, uint32_t fullX0, uint32_t empty0, int& n, int& st, bool& ok,
                                            unsigned char* qarea, float* xch, int pseg, int* pub_seq) {
    constexpr int KSTEPS = HD / 16, NTO = HD / 8, ROWB = HD * 2;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int Gq = a.Hq / a.Hkv, rows = a.att_rows, R = Gq * rows, base = a.att_base, total = base + rows;
    const uint32_t smem_base = smem_u32(smem);
    // ---- the queries come from the QKV phase: the activation producer's first arrival says it has finished
    if (ok) {
        ok = mbar_wait_err(fullX0 + 8 * st, (uint32_t)(n / kStages) & 1u, a.err);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok && lane == 0) atomicCAS(a.err, 0, 17000 + ph.layer);
    }
    uint4* qsm = reinterpret_cast<uint4*>(qarea);      // [k16 step][hi | lo][lane] A fragments of the 16 rows
    const float scale = rsqrtf((float)HD) * 1.4426950408889634f;   // scores in the log2 domain: p = 2^(s - m)
    for (int idx = threadIdx.x; idx < KSTEPS * 32; idx += kMegaEpiThreads) {
        const int ln = idx & 31, ks = idx >> 5, gg = ln >> 2, tt = ln & 3;
        float v[8];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int rho = gg + 8 * hh;
            float2 x0 = make_float2(0.f, 0.f), x1 = make_float2(0.f, 0.f);
            if (rho < R && ok) {
                const int gq = rho / rows, r = rho - gq * rows;
                const float* qp = a.q_out + ((size_t)r * a.Hq + kvh * Gq + gq) * HD + ks * 16 + 2 * tt;
                x0 = __ldcg(reinterpret_cast<const float2*>(qp));
                x1 = __ldcg(reinterpret_cast<const float2*>(qp + 8));
            }
            v[2 * hh] = x0.x * scale; v[2 * hh + 1] = x0.y * scale;
            v[4 + 2 * hh] = x1.x * scale; v[4 + 2 * hh + 1] = x1.y * scale;
        }
        uint16_t h[8], l[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) split_bf16(v[i], h[i], l[i]);
        qsm[(ks * 2 + 0) * 32 + ln] = make_uint4(pack2(h[0], h[1]), pack2(h[2], h[3]), pack2(h[4], h[5]), pack2(h[6], h[7]));
        qsm[(ks * 2 + 1) * 32 + ln] = make_uint4(pack2(l[0], l[1]), pack2(l[2], l[3]), pack2(l[4], l[5]), pack2(l[6], l[7]));
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");

    float o[NTO][4];
#pragma unroll
    for (int i = 0; i < NTO; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[i][e] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    int horizon[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const int rho = g + 8 * hh;
        horizon[hh] = rho < R ? base + rho % rows : -1;     // keys j <= horizon are visible (padding rows: unused)
    }
    int last_st = st;
    for (int tile = tile0; tile < tile1; ++tile, ++n) {
        if (ok) {
            const uint32_t par = (uint32_t)(n / kStages) & 1u;
            ok = mbar_wait_err(fullW0 + 8 * st, par, a.err) && mbar_wait_err(fullX0 + 8 * st, par, a.err);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok && lane == 0) atomicCAS(a.err, 0, 18000 + ph.layer);
        }
        const int j0 = tile * kAttTile + 8 * warp;           // first key of this warp's strip
        if (ok && j0 < total) {
            const uint32_t kst = smem_base + st * kStage, vst = kst + kAttTile * ROWB;
            const int row = 8 * warp + (lane & 7);
            if (j0 + 8 > total) {
                // rows beyond the keys hold whatever the pool or the stage held before: their probabilities are
                // exactly zero, but 0 x NaN is not, so their V rows are cleared (this warp's strip only)
                for (int i = lane; i < 8 * (ROWB / 16); i += 32) {
                    const int r = i / (ROWB / 16), cpos = i % (ROWB / 16);
                    if (j0 + r >= total)
                        *reinterpret_cast<uint4*>(smem + st * kStage + kAttTile * ROWB + (8 * warp + r) * ROWB + cpos * 16) =
                            make_uint4(0u, 0u, 0u, 0u);
                }
                __syncwarp();
            }
            // four independent accumulation chains (hi / lo terms x even / odd k16 steps), summed in a fixed order
            float s[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f}, s3[4] = {0.f, 0.f, 0.f, 0.f}, s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int kp = 0; kp < KSTEPS / 2; ++kp) {
                const uint4 qh0 = qsm[((2 * kp) * 2 + 0) * 32 + lane], ql0 = qsm[((2 * kp) * 2 + 1) * 32 + lane];
                const uint4 qh1 = qsm[((2 * kp + 1) * 2 + 0) * 32 + lane], ql1 = qsm[((2 * kp + 1) * 2 + 1) * 32 + lane];
                const int ch = kp * 4 + (lane >> 3);
                uint32_t b[4];
                ldsm_x4(b, kst + row * ROWB + ((ch ^ (row & 7)) << 4));
                mma_bf16_16816(s, qh0, b[0], b[1]);
                mma_bf16_16816(s2, ql0, b[0], b[1]);
                mma_bf16_16816(s3, qh1, b[2], b[3]);
                mma_bf16_16816(s4, ql1, b[2], b[3]);
            }
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int hh = e >> 1, j = j0 + 2 * t + (e & 1);
                s[e] = (s[e] + s3[e]) + (s2[e] + s4[e]);
                if (!(j < total && j <= horizon[hh])) s[e] = -INFINITY;
                mx[hh] = fmaxf(mx[hh], s[e]);
            }
            float alpha[2], m_use[2];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
                mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
                const float m_new = fmaxf(m_run[hh], mx[hh]);
                m_use[hh] = m_new == -INFINITY ? 0.f : m_new;      // keeps (-inf) - (-inf) out of the exponent
                alpha[hh] = ex2_approx(m_run[hh] - m_use[hh]);     // 0 while nothing has been seen yet
                m_run[hh] = m_new;
                l_run[hh] *= alpha[hh];
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                s[e] = ex2_approx(s[e] - m_use[e >> 1]);           // masked: 2^-inf = 0
                l_run[e >> 1] += s[e];                             // per-lane partial; the quad is summed at the end
            }
            if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
                for (int i = 0; i < NTO; ++i) {
                    o[i][0] *= alpha[0]; o[i][1] *= alpha[0];
                    o[i][2] *= alpha[1]; o[i][3] *= alpha[1];
                }
            }
            uint32_t ph0, pl0, ph1, pl1;
            split2(s[0], s[1], ph0, pl0);
            split2(s[2], s[3], ph1, pl1);
#pragma unroll
            for (int np = 0; np < NTO / 4; ++np) {
                const int ch = np * 4 + (lane >> 3);
                uint32_t b[4];
                ldsm_x4_trans(b, vst + row * ROWB + ((ch ^ (row & 7)) << 4));
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    mma_bf16_1688(o[4 * np + i], ph0, ph1, b[i]);
                    mma_bf16_1688(o[4 * np + i], pl0, pl1, b[i]);
                }
            }
        }
        last_st = st;
        if (tile + 1 < tile1) {      // the last tile's stage is kept: it is the merge's scratch
            asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
            if (threadIdx.x == 0 && ok) mbar_arrive(empty0 + 8 * st);
        }
        if (++st == kStages) st = 0;
    }
    // ---- merge the eight warps: common maximum, rescaled sums, outputs added in the order
    // ((w0 + w4) + (w1 + w5)) + (w2 + w6) + (w3 + w7)
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 1);
        l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 2);
    }
    float* ms = xch;            // [8 warps][16 rows] running maxima
    float* ls = xch + 128;      // [8 warps][16 rows] running sums
    if (t == 0) {
        ms[warp * 16 + g] = m_run[0]; ms[warp * 16 + g + 8] = m_run[1];
        ls[warp * 16 + g] = l_run[0]; ls[warp * 16 + g + 8] = l_run[1];
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
    float m_tot[2], l_tot[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const int row = g + 8 * hh;
        float m = -INFINITY, l = 0.f;
#pragma unroll
        for (int w = 0; w < kMegaEpiWarps; ++w) m = fmaxf(m, ms[w * 16 + row]);
#pragma unroll
        for (int w = 0; w < kMegaEpiWarps; ++w) {
            const float mw = ms[w * 16 + row];
            l += (mw == -INFINITY ? 0.f : exp2f(mw - m)) * ls[w * 16 + row];
        }
        const float sc = m_run[hh] == -INFINITY ? 0.f : exp2f(m_run[hh] - m);
#pragma unroll
        for (int i = 0; i < NTO; ++i) { o[i][2 * hh] *= sc; o[i][2 * hh + 1] *= sc; }
        m_tot[hh] = m;
        l_tot[hh] = l;
    }
    float* mo = reinterpret_cast<float*>(smem + last_st * kStage);      // [4][16 rows][HD]
    auto put = [&](int slot) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
            for (int i = 0; i < NTO; ++i)
                *reinterpret_cast<float2*>(mo + ((size_t)slot * 16 + g + 8 * hh) * HD + i * 8 + 2 * t) =
                    make_float2(o[i][2 * hh], o[i][2 * hh + 1]);
    };
    auto add = [&](int slot) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
            for (int i = 0; i < NTO; ++i) {
                const float2 v = *reinterpret_cast<const float2*>(mo + ((size_t)slot * 16 + g + 8 * hh) * HD + i * 8 + 2 * t);
                o[i][2 * hh] += v.x;
                o[i][2 * hh + 1] += v.y;
            }
    };
    if (warp >= 4) put(warp - 4);
    asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
    if (warp < 4) add(warp);
    asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
    if (warp >= 1 && warp < 4) put(warp);
    asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
    if (warp == 0) { add(1); add(2); add(3); }
    // warp 0 now holds the CTA's un-normalised output for the head, relative to m_tot, with the sum l_tot
    const int i0 = mega_owner(ub, T, G), i1 = mega_owner(ub + CPR - 1, T, G);
    constexpr int kSlotFloats = 8 * kMegaEpiThreads * 4;       // one CTA's slot of the exchange array
    if (i0 != i1 && cta != i0) {
        // contributor: output rows, maxima and sums to this CTA's slot; the publisher counts it in
        if (warp == 0) {
            float* dst = reinterpret_cast<float*>(a.scratch) + (size_t)cta * kSlotFloats;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                for (int i = 0; i < NTO; ++i)
                    *reinterpret_cast<float2*>(dst + (size_t)(g + 8 * hh) * HD + i * 8 + 2 * t) = make_float2(o[i][2 * hh], o[i][2 * hh + 1]);
                if (t == 0) { dst[16 * HD + g + 8 * hh] = m_tot[hh]; dst[16 * HD + 16 + g + 8 * hh] = l_tot[hh]; }
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
        if (threadIdx.x == 0) {
            fence_proxy_async_all();      // the stage served as scratch: ordinary stores before the next bulk copy into it
            if (ok) mbar_arrive(empty0 + 8 * last_st);
            st_release_cta(pub_seq, pseg);
        }
        return;
    }
    // collector (or alone on the head): own partial to shared memory, then all 256 threads finish the head
    if (warp == 0) {
        put(0);          // slot 0 of the scratch was last read by this warp itself
        if (t == 0) {
            ms[g] = m_tot[0]; ms[g + 8] = m_tot[1];
            ls[g] = l_tot[0]; ls[g + 8] = l_tot[1];
        }
    }
    if (i0 != i1 && threadIdx.x == 0) {
        const int n_contrib = T >= G ? i1 - i0 + 1 : CPR;
        if (!poll_counter(a.tickets + ph.ticket0 + kvh, n_contrib - 1, a.err)) atomicCAS(a.err, 0, 19000 + kvh);
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
    {
        constexpr int CPT = HD / 16;                            // output columns per thread
        const int row = threadIdx.x >> 4, c0 = (threadIdx.x & 15) * CPT;
        float num[CPT];
#pragma unroll
        for (int k = 0; k < CPT; ++k) num[k] = mo[(size_t)row * HD + c0 + k];
        float m = ms[row], den = ls[row];
        if (i0 != i1) {
            // contributions are fetched four CTAs at a time (all loads in flight) and merged in CTA order
            for (int ib = i0 + 1; ib <= i1; ib += 4) {
                float4 ov[4][CPT / 4];
                float mc[4], lc[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int i = ib + q;
                    const bool on = i <= i1 && (T >= G || mega_begin(i, T, G) != mega_begin(i + 1, T, G));
                    const float* src = reinterpret_cast<const float*>(a.scratch) + (size_t)i * kSlotFloats;
#pragma unroll
                    for (int k = 0; k < CPT / 4; ++k)
                        ov[q][k] = on ? __ldcg(reinterpret_cast<const float4*>(src + (size_t)row * HD + c0) + k)
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
                    mc[q] = on ? __ldcg(src + 16 * HD + row) : -INFINITY;
                    lc[q] = on ? __ldcg(src + 16 * HD + 16 + row) : 0.f;
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float mn = fmaxf(m, mc[q]);
                    const float wa = m == -INFINITY ? 0.f : exp2f(m - mn), wb = mc[q] == -INFINITY ? 0.f : exp2f(mc[q] - mn);
#pragma unroll
                    for (int k = 0; k < CPT / 4; ++k) {
                        num[4 * k] = num[4 * k] * wa + ov[q][k].x * wb;
                        num[4 * k + 1] = num[4 * k + 1] * wa + ov[q][k].y * wb;
                        num[4 * k + 2] = num[4 * k + 2] * wa + ov[q][k].z * wb;
                        num[4 * k + 3] = num[4 * k + 3] * wa + ov[q][k].w * wb;
                    }
                    den = den * wa + lc[q] * wb;
                    m = mn;
                }
            }
        }
        if (row < R && ok) {
            const int gq = row / rows, r = row - gq * rows;
            const float inv = 1.f / den;
#pragma unroll
            for (int k = 0; k < CPT; ++k) xu_store_one(ph.xf_out, r, (kvh * Gq + gq) * HD + c0 + k, num[k] * inv, NT);
        }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
    if (threadIdx.x == 0) {
        fence_proxy_async_all();
        if (ok) mbar_arrive(empty0 + 8 * last_st);
        st_release_cta(pub_seq, pseg);
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
    long long* kvoff_s = reinterpret_cast<long long*>(tail + 1536);   // [32] K/V slot offsets of the pass's rows
    int4* att_pg_s = reinterpret_cast<int4*>(tail + 1792);        // page ids of sixteen attention tiles (weight producer's)
    int* dep_seq = reinterpret_cast<int*>(tail + 328);            // 1 + last phase whose input is complete (activation producer -> epilogue)
    int* pub_seq = reinterpret_cast<int*>(tail + 320);            // segments whose stores are complete (epilogue -> publisher)
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
        *pub_seq = 0;
        *dep_seq = 0;
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
            MegaWalk ring;
            ring.start(a, cta, G);
            int n = 0, st = 0;
            bool ok = true;
            const uint64_t pol = l2_evict_first_policy();
            int att_phase = -1, att_c0 = 0;      // phase and first chunk whose page ids att_pg_s holds
            while (ring.valid()) {
                // At most kMegaMaxInFlight chunks are outstanding: enough to keep HBM busy (148 SMs x 96 KB is
                // twice the bandwidth-latency product), while every byte beyond that only queues in front of
                // the small latency-critical accesses of the phase boundaries (counters, partial sums, x).
                if (ok && n >= kMegaMaxInFlight) {
                    const int m = n - kMegaMaxInFlight;
                    ok = mbar_wait_err(fullW0 + 8 * (m % kStages), (uint32_t)(m / kStages) & 1u, a.err);
                }
                if (ok && n >= kStages) ok = mbar_wait_err(empty0 + 8 * st, (uint32_t)((n / kStages) - 1) & 1u, a.err);
                if (!ok) break;
                if (ring.mode == kPhaseAttn) {
                    // K/V tile of an attention phase: the pages cached before this pass (the others are the
                    // activation producer's).  Page ids are fetched sixteen tiles at a time (one memory latency
                    // per sixteen chunks instead of one per chunk) and kept in shared memory.
                    if (att_phase != ring.p || ring.c < att_c0 || ring.c >= att_c0 + 16) {
                        int4 tmp[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            tmp[i] = ring.c + i < ring.ce ? att_tile_pages(a, (ring.cc + i) % ring.CPR) : make_int4(0, 0, 0, 0);
#pragma unroll
                        for (int i = 0; i < 16; ++i) att_pg_s[i] = tmp[i];
                        att_phase = ring.p;
                        att_c0 = ring.c;
                    }
                    const int4 att_pages = att_pg_s[ring.c - att_c0];
                    const uint32_t bytes = att_issue_pages(a, ring.layer, ring.u, ring.cc, false, att_pages, 0, 0, true);
                    mbar_expect_tx(fullW0 + 8 * st, bytes);
                    att_issue_pages(a, ring.layer, ring.u, ring.cc, false, att_pages, smem_base + st * kStage, fullW0 + 8 * st, false);
                } else {
                    const uint32_t bytes = (uint32_t)ring.kc() * 4096u;
                    const bool two = ring.two();
                    mbar_expect_tx(fullW0 + 8 * st, two ? 2 * bytes : bytes);
                    bulk_g2s_hint(smem_base + st * kStage, ring.src(0), bytes, fullW0 + 8 * st, pol);
                    if (two) bulk_g2s_hint(smem_base + st * kStage + kMegaWHalf, ring.src(1), bytes, fullW0 + 8 * st, pol);
                }
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
    } else if (warp == kMegaWarpPub) {
        if (lane == 0) {
            // ---------------------------------------- publisher: walks the same schedule as the epilogue warps
            // and, whenever they have finished a segment (pub_seq), makes it known to the other CTAs: a
            // contribution counted in, or a unit counted as done.  The release (a fence over all the CTA's
            // earlier stores) costs a microsecond that no epilogue warp has to spend waiting.
            int seg = 0;
            bool ok = true;
            for (int p = a.p0; p < a.p1 && ok; ++p) {
                const MegaPhase& ph = a.phases[p];
                const int T = phase_chunks(a, ph), CPR = phase_cpr(a, ph);
                const int cb = mega_begin(cta, T, G), ce = mega_begin(cta + 1, T, G);
                int c = cb;
                while (c < ce) {
                    const int u = c / CPR, ub = u * CPR;
                    c = ce < ub + CPR ? ce : ub + CPR;
                    ++seg;
                    uint64_t t0 = 0;
                    for (uint32_t it = 0; ld_acquire_cta(pub_seq) < seg; ++it) {
                        __nanosleep(40);
                        if ((it & 63u) == 63u) {
                            if (ld_relaxed(a.err) != 0) { ok = false; break; }
                            const uint64_t now = global_ns();
                            if (t0 == 0) t0 = now;
                            else if (now - t0 > 4 * kMegaWaitNs) { ok = false; break; }
                        }
                    }
                    if (!ok) break;
                    const int i0 = mega_owner(ub, T, G), i1 = mega_owner(ub + CPR - 1, T, G);
                    if (i0 != i1 && cta != i0) red_release_add(a.tickets + ph.ticket0 + u, 1);
                    else red_release_add(a.done + p, 1);
                }
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
                if (lane == 0) {
                    ok = poll_counter(a.done + (p - 1), a.phases[p - 1].UB, a.err);
                    if (!ok) atomicCAS(a.err, 0, 12000 + p);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
            }
            if (!ok) break;
            if (lane == 0) st_release_cta(dep_seq, p + 1);
            if (p == a.p1 - 1) {
                // Successor kernels may be scheduled from here on -- but only once every CTA of this grid
                // is resident: a successor that took the place of a CTA still to come would wait for this
                // grid while this grid's phase boundaries wait for that CTA.
                if (lane == 0) ok = poll_counter(a.arrived, G, a.err);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                pdl_launch_dependents();
            }
            const int T = phase_chunks(a, ph), CPR = phase_cpr(a, ph), KS = ph.KS;
            const int cb = mega_begin(cta, T, G), ce = mega_begin(cta + 1, T, G);
            if (cb == ce) continue;
            if (lane == 0) {
                fence_proxy_async_all();          // activations were written with ordinary stores by other SMs
                const unsigned char* X = reinterpret_cast<const unsigned char*>(ph.xf);
                int cc = cb % CPR, u = cb / CPR;
                for (int c = cb; c < ce; ++c, ++n) {
                    if (n >= kStages) {
                        ok = mbar_wait_err(empty0 + 8 * st, (uint32_t)((n / kStages) - 1) & 1u, a.err);
                        if (!ok) break;
                    }
                    if (ph.mode == kPhaseAttn) {
                        // the pages of the tile that hold rows of this pass (written by the QKV phase); a tile
                        // without such pages still gets its arrival: the queries, too, come from that phase
                        uint32_t bytes = 0;
                        if ((cc + 1) * kAttTile > a.att_base) {
                            const int4 pages = att_tile_pages(a, cc);
                            bytes = att_issue_pages(a, ph.layer, u, cc, true, pages, 0, 0, true);
                            mbar_expect_tx(fullX0 + 8 * st, bytes);
                            att_issue_pages(a, ph.layer, u, cc, true, pages, smem_base + st * kStage, fullX0 + 8 * st, false);
                        } else {
                            mbar_expect_tx(fullX0 + 8 * st, 0u);
                        }
                    } else {
                        const int ks = cc * kMegaKC;
                        const int kc = KS - ks < kMegaKC ? KS - ks : kMegaKC;
                        const uint32_t bytes = (uint32_t)kc * NT * 512u;
                        mbar_expect_tx(fullX0 + 8 * st, bytes);
                        bulk_g2s(smem_base + st * kStage + kMegaWStage, X + (size_t)ks * NT * 512, bytes, fullX0 + 8 * st);
                    }
                    if (++st == kStages) st = 0;
                    if (++cc == CPR) { cc = 0; ++u; }
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
                const int T = phase_chunks(a, ph), CPR = phase_cpr(a, ph), KS = ph.KS, RB = ph.RB;
                const int cb = mega_begin(cta, T, G), ce = mega_begin(cta + 1, T, G);
                int c = cb;
                if (ph.mode == kPhaseAttn) {
                    // The attention chunks are consumed by the epilogue warps.  This thread still follows them
                    // one by one: a parity wait only tells the current barrier phase from the previous one, so
                    // a thread that skipped ahead by two uses of a stage would take an old phase for its own.
                    for (; c < ce; ++c, ++n) {
                        if (ok) {
                            const uint32_t par = (uint32_t)(n / kStages) & 1u;
                            ok = mbar_wait_err(fullW0 + 8 * st, par, a.err) && mbar_wait_err(fullX0 + 8 * st, par, a.err);
                            if (!ok) atomicCAS(a.err, 0, 13000 + p);
                        }
                        if (++st == kStages) st = 0;
                    }
                    continue;
                }
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
                            if (!ok) atomicCAS(a.err, 0, 13000 + p);
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
        if (threadIdx.x < 32) kvoff_s[threadIdx.x] = threadIdx.x < a.M ? a.row_kvoff[threadIdx.x] : 0;
        asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
        int seg = 0, n_norm = 0;      // n_norm: phases so far whose input is normalised and in which this CTA has work
        int pseg = 0;                 // segments finished (GEMM units and attention heads): what the publisher counts
        int n = 0, st = 0;            // chunk counter / ring stage: followed for the attention phases
        bool ok = true;
        const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * kCols);
        for (int p = a.p0; p < a.p1; ++p) {
            const MegaPhase& ph = a.phases[p];
            const int T = phase_chunks(a, ph), CPR = phase_cpr(a, ph), mode = ph.mode;
            const int cb = mega_begin(cta, T, G), ce = mega_begin(cta + 1, T, G);
            int c = cb;
            if (mode == kPhaseAttn) {
                while (c < ce) {
                    const int u = c / CPR, ub = u * CPR;
                    const int se = ce < ub + CPR ? ce : ub + CPR;
                    ++pseg;
                    if (a.hd == 128)
                        att_segment<128>(a, ph, p, cta, G, u, c - ub, se - ub, ub, T, CPR, NT, kStages, kStage, smem, fullW0, fullX0,
                                         empty0, n, st, ok, tail + kMegaTail, ssq_w, pseg, pub_seq);
                    else
                        att_segment<64>(a, ph, p, cta, G, u, c - ub, se - ub, ub, T, CPR, NT, kStages, kStage, smem, fullW0, fullX0,
                                        empty0, n, st, ok, tail + kMegaTail, ssq_w, pseg, pub_seq);
                    c = se;
                }
                continue;
            }
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
                const int buf = seg & 1;
                const int i0 = mega_owner(ub, T, G), i1 = mega_owner(ub + CPR - 1, T, G);
                float pa[MT], pb[MT];
                if (i0 == i1 || cta == i0) {      // this CTA runs the unit's epilogue: fetch its inputs now
                    // the residual stream is final once the phase's input is complete (it was written two phases
                    // back): the activation producer notes in dep_seq which phases' inputs it has seen complete
                    if (ok && mode == kResid) {
                        uint64_t t0 = 0;
                        for (uint32_t it = 0; ld_acquire_cta(dep_seq) <= p; ++it) {
                            if ((it & 63u) == 63u) {
                                const uint64_t now = global_ns();
                                if (t0 == 0) t0 = now;
                                else if (ld_relaxed(a.err) != 0 || now - t0 > kMegaWaitNs) { ok = false; break; }
                            }
                        }
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok && lane == 0) atomicCAS(a.err, 0, 20000 + p);
                    }
                    mega_preload<NT>(a, ph, u, warp, lane, pa, pb);
                }
                n += se - c;
                st = (st + (se - c)) % kStages;
                c = se;
                // A wait that gave up is not an exit: the warp keeps walking the schedule (without waiting) so
                // that it still meets the other epilogue warps at every named barrier below.
                if (ok) {
                    ok = mbar_wait_err(accfull0 + 8 * buf, (uint32_t)(seg >> 1) & 1u, a.err);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok && lane == 0) atomicCAS(a.err, 0, 15000 + p);
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
                ++pseg;
                // ---- the CTA's part of unit u is summed.  Alone on the unit: epilogue.  Otherwise the CTA that
                // owns the unit's first chunk collects (the unit is the last thing that CTA does in the phase,
                // so it waits for little): the others leave their rows in global memory and count themselves
                // in; the collector waits for that count, adds the contributions to its own in CTA order (a
                // fixed order), and runs the epilogue.  Contributors never wait.
                const int nq = (a.M + 3) / 4;           // 16-byte words of a row that hold real tokens
                if (i0 != i1) {
                    if (cta != i0) {
                        float4* mine = a.scratch + ((size_t)cta * (2 * NT)) * kMegaEpiThreads + threadIdx.x;
#pragma unroll
                        for (int q = 0; q < 2 * NT; ++q)
                            if (q < nq) mine[(size_t)q * kMegaEpiThreads] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                        // all stores of the CTA happen before thread 0's signal to the publisher thread (ordered by
                        // the named barrier), which counts the CTA in with a release
                        asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
                        if (threadIdx.x == 0) st_release_cta(pub_seq, pseg);
                        continue;
                    }
                    if (threadIdx.x == 0) {
                        // contributors: every CTA from i0 to i1 when each CTA owns at least one chunk; otherwise
                        // (fewer chunks than CTAs) every chunk of the unit belongs to a different CTA
                        const int n_contrib = T >= G ? i1 - i0 + 1 : CPR;
                        if (!poll_counter(a.tickets + ph.ticket0 + u, n_contrib - 1, a.err)) atomicCAS(a.err, 0, 14000 + p);
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
                    // contributions are fetched eight CTAs at a time, two 16-byte words each (16 loads in flight),
                    // and added in CTA order
                    for (int q0 = 0; q0 < 2 * NT; q0 += 2) {
                        if (q0 >= nq) break;
                        for (int ib = i0 + 1; ib <= i1; ib += 8) {
                            float4 w[8][2];
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const int i = ib + k;
                                const bool on = i <= i1 && (T >= G || mega_begin(i, T, G) != mega_begin(i + 1, T, G));
                                const float4* src = a.scratch + ((size_t)i * (2 * NT) + q0) * kMegaEpiThreads + threadIdx.x;
                                w[k][0] = on ? __ldcg(src) : make_float4(0.f, 0.f, 0.f, 0.f);
                                w[k][1] = (on && q0 + 1 < nq) ? __ldcg(src + kMegaEpiThreads) : make_float4(0.f, 0.f, 0.f, 0.f);
                            }
#pragma unroll
                            for (int k = 0; k < 8; ++k)
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    v[4 * (q0 + h)] += w[k][h].x;
                                    v[4 * (q0 + h) + 1] += w[k][h].y;
                                    v[4 * (q0 + h) + 2] += w[k][h].z;
                                    v[4 * (q0 + h) + 3] += w[k][h].w;
                                }
                        }
                    }
                }
                if (mode == kPlain) mega_epilogue<NT, kPlain>(a, ph, p, cta, u, warp, lane, v, pa, pb, rstd_s, ssq_w, kvoff_s);
                else if (mode == kQkvRope) mega_epilogue<NT, kQkvRope>(a, ph, p, cta, u, warp, lane, v, pa, pb, rstd_s, ssq_w, kvoff_s);
                else if (mode == kResid) mega_epilogue<NT, kResid>(a, ph, p, cta, u, warp, lane, v, pa, pb, rstd_s, ssq_w, kvoff_s);
                else mega_epilogue<NT, kSwiglu>(a, ph, p, cta, u, warp, lane, v, pa, pb, rstd_s, ssq_w, kvoff_s);
                // publish: the named barrier orders every thread's stores before thread 0's signal; the publisher
                // thread counts the unit as done with a release, so that no epilogue warp waits for the fence;
                // readers acquire the counter (and fence the asynchronous proxy before their bulk copies)
                asm volatile("bar.sync 1, %0;" ::"n"(kMegaEpiThreads) : "memory");
                if (threadIdx.x == 0) st_release_cta(pub_seq, pseg);
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
