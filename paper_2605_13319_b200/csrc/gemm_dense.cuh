// Dense weight-streaming GEMM for passes of more than 32 rows (a batch of requests, a prefill chunk):
// y[M,N] = x[M,K] . W[N,K]^T on the tcgen05 tensor cores, with the same fused epilogues as the small-M kernel.
//
// One CTA = one 128-row block of W x one token block of up to 160 tokens x the whole of K: no split-K, so a
// result element is summed in one fixed order (k ascending; within a k16 step the bf16 hi term, then the lo term)
// whatever the batch, and every weight byte is read once per token block.  The weight tile is the M = 128 side of
// the MMA (A operand, K-major, packed at context creation in the operand's own core-matrix order); the tokens are
// the N side (B operand): activations arrive as split-bf16 hi and lo tiles in operand order ("xd" arrays, written
// by the producing kernel's epilogue), two MMAs per k16 step into one fp32 accumulator in tensor memory
// (128 lanes = weight rows, one column per token).
// Two CTAs share an SM (half of its shared memory and tensor memory each), so that one's epilogue runs under the
// other's main loop.
// Warp 0: one lane streams (weights, activations) chunks into a shared-memory ring with bulk copies (weights before
// the dependent-launch wait).  Warp 1: one lane issues the MMAs; tcgen05.commit frees a ring stage / hands the
// accumulator over.  Warps 2-5: the input's RMSNorm factors while the ring streams, then the epilogue: tcgen05.ld
// (thread = weight row, registers = 16 tokens at a time) and the mode's arithmetic.
#pragma once
#include "common.cuh"
#include "gemm.cuh"
#include "tcgen05.cuh"

namespace pipesd {

constexpr int kDenseThreads = 192;
constexpr int kDenseEpi = 128;            // threads of warps 2-5
constexpr int kDenseMaxTok = 160;         // tokens per CTA: columns of the accumulator (a multiple of 16)
constexpr int kDenseMaxStages = 7;
constexpr int kDenseTail = 128 + 4 * kDenseMaxTok + 4 * 4 * 16;   // barriers, tensor-memory base | rstd[160] | sums of squares [4 warps][16]
constexpr int kDenseSmemHalf = (228 * 1024) / 2 - 1024;          // dynamic shared memory of a CTA when two share an SM
constexpr int kDenseSmemWhole = 227 * 1024;                      // ... when it has the SM to itself
static_assert(8 * (2 * kDenseMaxStages + 1) + 4 <= 128, "barriers and the tensor-memory slot fill the first 128 bytes of the tail");

// ---- weights in tensor-core operand order --------------------------------------------------------------------
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

// ---- "xd" activation arrays: the K-major B operand of tcgen05.mma, in global memory ---------------------------
// Token blocks of TBS tokens (a multiple of 16).  Per (token block, k16 step): the bf16 hi tile then the lo tile,
// TBS * 32 bytes each, cut into 8x8 core matrices: element (token t, k) of a tile at
// ((t / 8) * 2 + (k / 8) % 2) * 128 + (t % 8) * 16 + (k % 8) * 2.  A chunk of consecutive k16 steps of a token block
// is one contiguous run.  (xd_store_one and act_store_one, next to the fragment-order stores, write these.)
struct XdPlan { int tbs, n_tb; };          // tokens per block, blocks
// Host: the token blocks of a GEMM with N output rows over M tokens on a device of n_sm SMs.  The tensor cores bound
// the kernel: an SM's time is about (CTAs it runs) x (a per-step cost that grows with the tokens of a block: fetch of
// the weight tile + fetch of and product with the token tile), so the plan is the block count that minimises
// ceil(CTAs / n_sm) x (32 + 3/4 tokens per block) -- few, large blocks unless they leave SMs idle or a last wave nearly
// empty; the fewest blocks among equals.  A function of (M, N, n_sm) alone: producer and consumer derive the same plan.
static inline XdPlan dense_plan(int M, int N, int n_sm) {
    const int RB = (N + 127) / 128;
    const int lo = (M + kDenseMaxTok - 1) / kDenseMaxTok, hi = (M + 15) / 16;
    XdPlan best = {kDenseMaxTok, lo < 1 ? 1 : lo};
    double best_cost = 1e300;
    for (int n = lo < 1 ? 1 : lo; n <= hi && n <= lo + 16; ++n) {
        const int tbs = ((M + n - 1) / n + 15) / 16 * 16;
        const int n_tb = (M + tbs - 1) / tbs;
        const double cost = (double)((RB * n_tb + n_sm - 1) / n_sm) * (32.0 + 0.75 * tbs);
        if (cost < best_cost - 1e-9) { best_cost = cost; best.tbs = tbs; best.n_tb = n_tb; }
    }
    return best;
}
// Host: the ring of a launch of `ctas` CTAs.  More CTAs than SMs: two per SM, each with half of the shared memory
// and stages of two k16 steps; otherwise a CTA has its SM to itself and keeps twice the bytes in flight.
struct DenseRing { int kc, stages; size_t smem; };
static inline DenseRing dense_ring(int tbs, int ctas, int n_sm) {
    DenseRing r;
    const bool whole = ctas <= n_sm;
    r.kc = whole ? 4 : 2;
    const int stage = r.kc * (4096 + tbs * 64);
    const int s = ((whole ? kDenseSmemWhole : kDenseSmemHalf) - kDenseTail) / stage;
    r.stages = s > kDenseMaxStages ? kDenseMaxStages : s;
    r.smem = (size_t)r.stages * stage + kDenseTail;
    return r;
}
__host__ __device__ constexpr int dense_tmem_cols(int tbs) {
    int c = 32;
    while (c < tbs) c *= 2;
    return c;
}

struct DenseArgs {
    GemmArgs g;         // W = weights in operand order; xf = input xd array; the mode's outputs as for the small-M kernel
    int kc;             // k16 steps per ring stage (g.stages stages)
    int tbs_in;         // token block size of the input array and of this launch
    int tbs_out;        // token block size of the xd array this launch produces (kResid, kSwiglu)
};

// grid (128-row blocks, token blocks), block 192.  The bound of 256 threads x 2 CTAs caps a thread at 128 registers:
// a CTA's six warps put two on one register partition of the SM (a quarter of the register file), and two CTAs must
// fit there side by side.
template <int MODE>
__global__ void __launch_bounds__(256, 2) gemm_dense_kernel(const DenseArgs da) {
    const GemmArgs& a = da.g;
    extern __shared__ __align__(128) unsigned char smem[];
    const int TBS = da.tbs_in;
    const int KC = da.kc;
    const int w_stage = KC * 4096, b_stage = KC * TBS * 64;
    const int stage_bytes = w_stage + b_stage;
    const int stages = a.stages;
    unsigned char* tail = smem + stages * stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);                // full[7], empty[7], acc_full
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 8 * (2 * kDenseMaxStages + 1));
    float* rstd_s = reinterpret_cast<float*>(tail + 128);              // [TBS]
    float* ssq_s = rstd_s + kDenseMaxTok;                              // [4 warps][16 tokens]
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kDenseMaxStages, acc_full = full0 + 16 * kDenseMaxStages;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rb = blockIdx.x, tb = blockIdx.y;
    const int KS = a.KS, nchunks = (KS + KC - 1) / KC;
    const int tok0 = tb * TBS;
    const uint32_t tmem_cols = (uint32_t)dense_tmem_cols(TBS);

    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, 1);
        }
        mbar_init(acc_full, 1);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), tmem_cols);
        tc_fence_before();
    }
    __syncthreads();
    pdl_launch_dependents();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

    bool ok = true;
    if (warp == 0) {
        // ---------------- producer: lane 0 streams (weights, activations) chunks into the ring
        if (lane == 0) {
            const unsigned char* wsrc = reinterpret_cast<const unsigned char*>(a.W) + (size_t)rb * KS * 4096;
            const unsigned char* bsrc = reinterpret_cast<const unsigned char*>(a.xf) + (size_t)tb * KS * (TBS * 64);
            auto chunk_ks = [&](int c) { int r = KS - c * KC; return r < KC ? r : KC; };
            const int pre = nchunks < stages ? nchunks : stages;
            const uint64_t pol = l2_evict_first_policy();
            // weights do not depend on the previous kernel: start them before the dependency wait
            for (int c = 0; c < pre; ++c) {
                const int kc = chunk_ks(c);
                mbar_expect_tx(full0 + 8 * c, (uint32_t)kc * (4096 + TBS * 64));
                bulk_g2s_hint(smem_base + c * stage_bytes, wsrc + (size_t)c * w_stage, (uint32_t)kc * 4096, full0 + 8 * c, pol);
            }
            pdl_wait();
            for (int c = 0; c < pre; ++c) {
                const int kc = chunk_ks(c);
                bulk_g2s(smem_base + c * stage_bytes + w_stage, bsrc + (size_t)c * b_stage, (uint32_t)kc * TBS * 64, full0 + 8 * c);
            }
            int issued = pre, st = 0;
            uint32_t ph = 0;
            for (int c = pre; c < nchunks; ++c) {
                const int kc = chunk_ks(c);
                ok = mbar_wait(empty0 + 8 * st, ph);
                if (!ok) break;
                mbar_expect_tx(full0 + 8 * st, (uint32_t)kc * (4096 + TBS * 64));
                bulk_g2s_hint(smem_base + st * stage_bytes, wsrc + (size_t)c * w_stage, (uint32_t)kc * 4096, full0 + 8 * st, pol);
                bulk_g2s(smem_base + st * stage_bytes + w_stage, bsrc + (size_t)c * b_stage, (uint32_t)kc * TBS * 64, full0 + 8 * st);
                issued = c + 1;
                if (++st == stages) { st = 0; ph ^= 1u; }
            }
            if (!ok) {
                if (a.err) atomicExch(a.err, 6);
                // give up: let every copy already issued land before this CTA's shared memory is released
                for (int c = issued > stages ? issued - stages : 0; c < issued; ++c)
                    mbar_wait(full0 + 8 * (c % stages), (c / stages) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(128, TBS, 0, 0);
            int st = 0;
            uint32_t ph = 0;
            for (int c = 0; c < nchunks; ++c) {
                ok = mbar_wait(full0 + 8 * st, ph);
                if (!ok) break;
                tc_fence_after();
                const uint32_t wst = smem_base + st * stage_bytes, bst = wst + w_stage;
                int kc = KS - c * KC;
                kc = kc < KC ? kc : KC;
                for (int k = 0; k < kc; ++k) {
                    const uint64_t ad = umma_desc(wst + k * 4096, 128, 256);
                    umma_bf16(tmem, ad, umma_desc(bst + (k * 2) * TBS * 32, 128, 256), idesc, (c > 0 || k > 0) ? 1u : 0u);
                    umma_bf16(tmem, ad, umma_desc(bst + (k * 2 + 1) * TBS * 32, 128, 256), idesc, 1u);
                }
                umma_commit(empty0 + 8 * st);      // the stage is free when these MMAs have read it
                if (++st == stages) { st = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(acc_full);
            else if (a.err) atomicExch(a.err, 7);
        }
    } else {
        // ---------------- epilogue warps: thread = weight row (tensor-memory lane 32 * (warp % 4) + lane)
        const int et = threadIdx.x - 64;                               // 0..127
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;                           // row within the block
        const int pr = rb * 128 + row;                                 // packed row
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        pdl_wait();
        if (a.ssq_in != nullptr) {
            for (int tl = et; tl < TBS; tl += kDenseEpi) {
                const int tok = tok0 + tl;
                float ss = 0.f;
                if (tok < a.M)
                    for (int b = 0; b < a.n_ssq; ++b) ss += a.ssq_in[(size_t)b * a.M + tok];
                rstd_s[tl] = rsqrtf(ss / (float)a.d_in + a.eps);
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kDenseEpi) : "memory");
        // per-row constants of the mode
        float gain = 0.f;
        if (MODE == kResid && pr < a.N) gain = a.gain_next[pr];
        const int half_hd = a.hd / 2;
        int lr = 0, head = 0, dim = 0;
        if (MODE == kQkvRope) { lr = qkv_logical_row(pr, a.hd); head = lr / a.hd; dim = lr % a.hd; }
        ok = mbar_wait(acc_full, 0);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        const bool row_live = pr < a.N;
        const int prc = row_live ? pr : a.N - 1;
        // the activation output: this thread's column of the consumer's xd array; a 16-token column block of the
        // accumulator lies inside one of its token blocks (block sizes and block starts are multiples of 16)
        const int k_out = MODE == kSwiglu ? gu_feature(prc) : prc;
        const int KS_out = (MODE == kSwiglu ? a.N / 2 : a.N) / 16;
        uint16_t* act_out = MODE == kSwiglu ? a.xf_act : a.xf_out;
        const uint32_t ocol = act_index_col(k_out, 0, da.tbs_out), olo = act_index_lo(da.tbs_out);
        for (int cb = 0; cb < TBS / 16; ++cb) {
            float v[16];
            tmem_ld16(tmem + lane_sel + cb * 16, v);
            // what the mode reads per element, fetched for the 16 tokens at once (independent loads, clamped addresses)
            // while the accumulator columns arrive
            float e0[16], e1[16];
            long long rk[16];
            if (MODE == kResid) {
#pragma unroll
                for (int i = 0; i < 16; ++i) e0[i] = a.x[(size_t)min(tok0 + cb * 16 + i, a.M - 1) * a.N + prc];
            } else if (MODE == kQkvRope) {
                const bool rot = head < a.Hq + a.Hkv, cached = head >= a.Hq;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int tokc = min(tok0 + cb * 16 + i, a.M - 1);
                    e0[i] = rot ? a.cs[(size_t)tokc * half_hd + (dim % half_hd)] : 1.f;
                    e1[i] = rot ? a.sn[(size_t)tokc * half_hd + (dim % half_hd)] : 0.f;
                    rk[i] = cached ? a.row_kvoff[tokc] : 0;
                }
            }
            const uint32_t orow = (MODE == kResid || MODE == kSwiglu) ? act_index_row(tok0 + cb * 16, 0, KS_out, 0, da.tbs_out) + ocol : 0u;
            tmem_ld_wait();
            float sq[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int tl = cb * 16 + i, tok = tok0 + tl;
                float x = ok ? v[i] : 0.f;
                if (a.ssq_in != nullptr) x *= rstd_s[tl];
                const bool live = tok < a.M && row_live;
                sq[i] = 0.f;
                if (MODE == kPlain) {
                    if (live) a.out[(size_t)tok * a.N + pr] = x;
                } else if (MODE == kResid) {
                    float xn = 0.f;
                    if (live) {
                        xn = e0[i] + x;
                        a.x[(size_t)tok * a.N + pr] = xn;
                        act_store_at(act_out, orow + (uint32_t)((i >> 3) * 128 + (i & 7) * 8), olo, xn * gain);
                    }
                    sq[i] = xn * xn;
                } else {
                    // both remaining modes pair row i (< 8) with row i + 8 of a 16-row tile
                    const float partner = __shfl_xor_sync(0xffffffffu, x, 8);
                    if (MODE == kSwiglu) {
                        if ((row & 15) < 8 && live) {
                            const float act = x / (1.f + expf(-x)) * partner;      // own = gate, partner = up
                            act_store_at(act_out, orow + (uint32_t)((i >> 3) * 128 + (i & 7) * 8), olo, act);
                        }
                    } else if (live) {                                           // kQkvRope
                        // q and k heads are rotated (cos = 1, sin = 0 for v heads)
                        const float val = (row & 15) < 8 ? x * e0[i] - partner * e1[i] : x * e0[i] + partner * e1[i];
                        if (head < a.Hq) {
                            a.q_out[((size_t)tok * a.Hq + head) * a.hd + dim] = val;
                        } else {
                            const int kv = head < a.Hq + a.Hkv ? 0 : 1;
                            const int kvh = kv ? head - a.Hq - a.Hkv : head - a.Hq;
                            const size_t per_head = (size_t)a.page_size * a.hd;
                            const size_t off = (size_t)a.layer * a.n_pages * 2 * a.Hkv * per_head + (size_t)rk[i] +
                                               ((size_t)kv * a.Hkv + kvh) * per_head + kv_col_offset(dim);
                            a.kv_pool[off] = f32_to_bf16_bits(val);
                        }
                    }
                }
            }
            if (MODE == kResid) {
                // sums of squares of the new rows over the block's 128 rows, per token: over the warp's 32 rows by
                // recursive halving (lane i ends up with token i's sum, lanes 16-31 mirror 0-15), then over the four
                // warps in order
#pragma unroll
                for (int w = 8; w >= 1; w >>= 1) {
                    const bool upper = (lane & w) != 0;
#pragma unroll
                    for (int i = 0; i < w; ++i) {
                        const float keep = upper ? sq[i + w] : sq[i], give = upper ? sq[i] : sq[i + w];
                        sq[i] = keep + __shfl_xor_sync(0xffffffffu, give, w);
                    }
                }
                sq[0] += __shfl_xor_sync(0xffffffffu, sq[0], 16);
                if (lane < 16) ssq_s[quarter * 16 + lane] = sq[0];       // lane l: token l of the column block
                asm volatile("bar.sync 1, %0;" ::"n"(kDenseEpi) : "memory");
                if (et < 16) {
                    const int tl = cb * 16 + et, tok = tok0 + tl;
                    if (tok < a.M)
                        a.ssq_out[(size_t)rb * a.M + tok] = ssq_s[et] + ssq_s[16 + et] + ssq_s[32 + et] + ssq_s[48 + et];
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kDenseEpi) : "memory");
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, tmem_cols);
    }
}

}  // namespace pipesd
