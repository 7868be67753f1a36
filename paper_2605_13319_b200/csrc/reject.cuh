// Vocabulary-wide part of the verify pass: row softmax statistics, the sequential accept chain, and
// the single final draw (residual resample on a rejection, extra token when all drafts pass).
//
// Rule: accept draft x_i while u_i < min(1, p_i(x_i) / q_i(x_i)); on the first failure at row r draw
// the correction from norm(max(0, p_r - q_r)); when all k pass draw the extra token from p_k.
// Greedy mode: accept while the draft is the row's argmax (lowest index on ties), emit the argmax.
// Decisions are taken in fp64 on fp32 logits; sums run in a fixed order, so a result is reproducible.
#pragma once
#include "common.cuh"

namespace pipesd {

constexpr int kStatSplits = 16;     // column splits per row in the statistics kernel
constexpr int kSampleThreads = 1024;

struct RowStat {
    float m;       // max logit in the split
    int arg;       // its lowest index
    double z;      // sum exp(l - m) over the split
};

// Per (row, split) of the logits: max, argmax, sum-exp.  grid (M, kStatSplits), block 256.
__global__ void __launch_bounds__(256) row_stats_kernel(int V, const float* __restrict__ logits,
                                                        RowStat* __restrict__ stats) {
    const int row = blockIdx.x, sp = blockIdx.y;
    const int per = (V + kStatSplits - 1) / kStatSplits;
    const int j0 = sp * per, j1 = min(V, j0 + per);
    const float* lr = logits + (size_t)row * V;
    float m = -INFINITY;
    int arg = 0x7fffffff;
    for (int j = j0 + threadIdx.x; j < j1; j += 256) {
        const float v = lr[j];
        if (v > m) { m = v; arg = j; }
    }
    __shared__ float sm_m[8];
    __shared__ int sm_a[8];
    __shared__ double sm_z[8];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float om = __shfl_xor_sync(0xffffffffu, m, o);
        int oa = __shfl_xor_sync(0xffffffffu, arg, o);
        if (om > m || (om == m && oa < arg)) { m = om; arg = oa; }
    }
    if ((threadIdx.x & 31) == 0) { sm_m[threadIdx.x >> 5] = m; sm_a[threadIdx.x >> 5] = arg; }
    __syncthreads();
    m = sm_m[0]; arg = sm_a[0];
#pragma unroll
    for (int w = 1; w < 8; ++w)
        if (sm_m[w] > m || (sm_m[w] == m && sm_a[w] < arg)) { m = sm_m[w]; arg = sm_a[w]; }
    double z = 0.0;
    for (int j = j0 + threadIdx.x; j < j1; j += 256) z += (double)expf(lr[j] - m);
    z = warp_sum_d(z);
    if ((threadIdx.x & 31) == 0) sm_z[threadIdx.x >> 5] = z;
    __syncthreads();
    if (threadIdx.x == 0) {
        double zt = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) zt += sm_z[w];
        RowStat st;
        st.m = m; st.arg = arg; st.z = zt;
        stats[(size_t)row * kStatSplits + sp] = st;
    }
}

struct RejectItem {
    int row0;          // first logits row of the request
    int k;             // drafts
    int mode;          // 0 stochastic, 1 greedy, 2 none (prefill)
    int u0;            // offset of the request's k+1 uniforms
    const float* q;    // device [k][V]
    int slot;          // request slot (row of the request-state array)
    int base;          // cached positions before this pass, as the host planned it
    int commit;        // kCommit*: what the kernel does with the request's device-resident state
    int reserved;
};

struct RejectOut { int n_accepted, next_token, status, reserved; };

// Device-resident request state, kept by the commit-on-device path: the committed length and the pending token
// (the last correction or extra token, whose K/V is not cached yet), and whether the last pass accepted every draft.
struct ReqState { int len, pending, all_accepted, reserved; };
constexpr int kCommitNone = 0;      // the host commits later (pipesd_kv_rollback)
constexpr int kCommitAuto = 1;      // write {base + 1 + n_accepted, emitted token} to the state
constexpr int kCommitChain = 2;     // as kCommitAuto, but only if the state says that the pass before this one accepted every
                                    // draft, left exactly `base` positions and emitted this pass's first token
                                    // (early drafts kept by the cloud are valid under exactly that condition); otherwise the pass
                                    // is void: status kStatusDiscarded, state untouched apart from all_accepted = 0
constexpr int kStatusDiscarded = 1;

// One CTA per request: combine the row statistics, run the accept chain, make the final draw.
//
// Accept chain: the k ratio tests are independent of each other (only "stop at the first failure" is sequential),
// so thread i evaluates test i and thread 0 takes the first failure.
// Final draw, inverse CDF in token-id order, by a cluster of kSampleCluster CTAs per request: warp w of CTA r owns
// the contiguous ids [(r * warps + w) * R, ... + R) (R a multiple of 32) and walks them 32 at a time, lane = id, so
// that every load is coalesced and the fp64 exponentials of a vocabulary-wide row are spread over eight SMs.
// Pass 1 adds each lane's terms in walk order and the lanes in butterfly order (fixed); a CTA scans its warp totals
// in warp order, the CTA totals cross the cluster once (every CTA adds them up in rank order, so all of them hold
// the same prefixes bit for bit).  Pass 2 runs only in the one warp whose range holds the target: an inclusive
// shuffle scan per 32 ids on top of the running prefix, the first id whose prefix exceeds u * total wins.
constexpr int kSampleCluster = 8;
__device__ __forceinline__ void dsmem_st_f64(uint32_t addr, double v) {
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}

// grid (kSampleCluster, n_items), cluster (kSampleCluster, 1, 1).
__global__ void __launch_bounds__(kSampleThreads) accept_sample_kernel(const float* __restrict__ logits, int V,
                                                                       const RowStat* __restrict__ stats,
                                                                       const RejectItem* __restrict__ items,
                                                                       const int32_t* __restrict__ row_tok,
                                                                       const float* __restrict__ u_all,
                                                                       RejectOut* __restrict__ out,
                                                                       ReqState* __restrict__ req_state) {
    pdl_wait();      // launched with programmatic serialisation: the row statistics must be complete
    const int item = blockIdx.y, rank = (int)cluster_ctarank();
    const RejectItem it = items[item];
    if (it.mode == 2) return;                     // the whole cluster (one request) leaves together
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (it.commit == kCommitChain) {
        // the state was written by the pass before this one (an earlier launch): every thread reads the same values
        const ReqState s = req_state[it.slot];
        if (!(s.all_accepted && s.len == it.base && s.pending == row_tok[it.row0])) {
            if (rank == 0 && tid == 0) {
                RejectOut r{0, -1, kStatusDiscarded, 0};
                out[item] = r;
                req_state[it.slot].all_accepted = 0;
            }
            return;
        }
    }
    // exactly one thread of the cluster publishes the result and, on the commit-on-device path, the new state
    auto emit = [&](int n_acc_, int tok_) {
        RejectOut r{n_acc_, tok_, 0, 0};
        out[item] = r;
        if (it.commit != kCommitNone) {
            ReqState s{it.base + 1 + n_acc_, tok_, n_acc_ == it.k ? 1 : 0, 0};
            req_state[it.slot] = s;
        }
    };
    constexpr int kWarps = kSampleThreads / 32;
    __shared__ double s_m[kMaxItemRows], s_z[kMaxItemRows];
    __shared__ int s_arg[kMaxItemRows];
    __shared__ int s_ok[kMaxItemRows];
    __shared__ int s_nacc;
    __shared__ double s_warp[kWarps];      // warp totals, then their exclusive prefixes
    __shared__ double s_incl[kWarps];      // inclusive prefixes of the warp totals
    __shared__ double s_total, s_base;
    __shared__ double s_cta[2][kSampleCluster];   // the CTAs' totals, written by their owners; one set per attempt

    if (tid <= it.k) {   // rows 0..k: merge the column splits
        const RowStat* st = stats + (size_t)(it.row0 + tid) * kStatSplits;
        float m = st[0].m;
        int arg = st[0].arg;
        for (int s = 1; s < kStatSplits; ++s)
            if (st[s].m > m || (st[s].m == m && st[s].arg < arg)) { m = st[s].m; arg = st[s].arg; }
        double z = 0.0;
        for (int s = 0; s < kStatSplits; ++s)
            if (st[s].m > -INFINITY) z += st[s].z * exp((double)st[s].m - (double)m);
        s_m[tid] = (double)m; s_z[tid] = z; s_arg[tid] = arg;
    }
    __syncthreads();
    if (tid < it.k) {    // test i: draft i+1 against row i
        const int x = row_tok[it.row0 + tid + 1];
        bool ok;
        if (it.mode == 1) {
            ok = (x == s_arg[tid]);
        } else {
            const double p = exp((double)logits[(size_t)(it.row0 + tid) * V + x] - s_m[tid]) / s_z[tid];
            const double qx = (double)it.q[(size_t)tid * V + x];
            const double ratio = qx > 0.0 ? p / qx : (p > 0.0 ? INFINITY : 0.0);
            ok = (double)u_all[it.u0 + tid] < fmin(ratio, 1.0);
        }
        s_ok[tid] = ok ? 1 : 0;
    }
    __syncthreads();
    if (tid == 0) {
        int n = 0;
        while (n < it.k && s_ok[n]) ++n;
        s_nacc = n;
    }
    __syncthreads();
    const int n_acc = s_nacc;
    if (it.mode == 1) {
        if (tid == 0 && rank == 0) emit(n_acc, s_arg[n_acc]);
        return;
    }
    // Final draw from row n_acc: residual max(0, p - q) if a draft was rejected there, else p.
    const float* lr = logits + (size_t)(it.row0 + n_acc) * V;
    const double m = s_m[n_acc], inv_z = 1.0 / s_z[n_acc];
    const double uk = (double)u_all[it.u0 + it.k];
    constexpr int kAllWarps = kSampleCluster * kWarps;
    const int R = ((V + kAllWarps - 1) / kAllWarps + 31) / 32 * 32;     // ids per warp
    const int j0 = min(V, (rank * kWarps + warp) * R), j1 = min(V, j0 + R);
    bool use_q = n_acc < it.k;
    const float* qr = use_q ? it.q + (size_t)n_acc * V : nullptr;
    auto term = [&](int j) -> double {
        if (j >= j1) return 0.0;
        double r = exp((double)lr[j] - m) * inv_z;
        if (use_q) r = fmax(0.0, r - (double)qr[j]);
        return r;
    };
    for (int attempt = 0; attempt < 2; ++attempt) {
        double loc = 0.0;
        for (int j = j0 + lane; j < j1; j += 32) loc += term(j);
        const double wsum = warp_sum_d(loc);
        if (lane == 0) s_warp[warp] = wsum;
        __syncthreads();
        if (warp == 0) {
            double w = s_warp[lane], winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                double t = __shfl_up_sync(0xffffffffu, winc, o);
                if (lane >= o) winc += t;
            }
            double excl = __shfl_up_sync(0xffffffffu, winc, 1);
            if (lane == 0) excl = 0.0;
            s_warp[lane] = excl;         // exclusive prefix of the warp totals = the previous warp's inclusive one, exactly
            s_incl[lane] = winc;
            const double cta_total = __shfl_sync(0xffffffffu, winc, 31);
            if (lane < kSampleCluster)   // this CTA's total into every CTA's table
                dsmem_st_f64(dsmem_addr(smem_u32(&s_cta[attempt][rank]), (uint32_t)lane), cta_total);
        }
        cluster_sync_all();
        if (tid == 0) {
            double run = 0.0, base = 0.0;
            for (int r = 0; r < kSampleCluster; ++r) {
                if (r == rank) base = run;
                run += s_cta[attempt][r];
            }
            s_base = base;               // ranks before this one, added in rank order: equals the previous CTA's
            s_total = run;               // base + total exactly, so the prefixes are monotone across CTAs as well
        }
        __syncthreads();
        const double total = s_total;
        if (use_q && !(total > 0.0)) {   // p <= q everywhere (e.g. p == q): fall back to p
            use_q = false;
            __syncthreads();
            continue;
        }
        const double target = uk * total;
        // the owner is the first warp whose inclusive prefix exceeds the target (warp-uniform test)
        const double before = s_base + s_warp[warp];
        const bool mine = s_base + s_incl[warp] > target && !(before > target);     // exactly one warp of the cluster
        if (mine) {
            double run = before;
            int tok = -1, last_mass = -1;
            for (int c = j0; c < j1 && tok < 0; c += 32) {
                double inc = term(c + lane);
                const unsigned mass = __ballot_sync(0xffffffffu, inc > 0.0);
                if (mass) last_mass = c + 31 - __clz(mass);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    double t = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += t;
                }
                const unsigned hit = __ballot_sync(0xffffffffu, run + inc > target && c + lane < j1);
                if (hit) tok = c + __ffs(hit) - 1;
                run += __shfl_sync(0xffffffffu, inc, 31);
            }
            if (tok < 0) tok = last_mass;    // the walk's rounding fell short of the range's total: its last id with mass
            if (lane == 0) emit(n_acc, tok);
        }
        // u < 1, so target < total and some warp owns it; were rounding ever to say otherwise, rank 0 answers
        if (!(total > target) && rank == 0 && tid == 0) {
            // target >= every prefix (rounding at the top of the CDF): last token with mass
            int tok = V - 1;
            for (int j = V - 1; j >= 0; --j) {
                double r = exp((double)lr[j] - m) * inv_z;
                if (use_q) r = fmax(0.0, r - (double)qr[j]);
                if (r > 0.0) { tok = j; break; }
            }
            emit(n_acc, tok);
        }
        break;
    }
}

}  // namespace pipesd
