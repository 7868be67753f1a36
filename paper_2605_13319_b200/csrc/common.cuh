// Shared device helpers for the NAV verify kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pipesd {

constexpr int kMaxItemRows = 32;   // rows (k+1, or a prefill chunk) one request contributes to a pass
constexpr int kMaxSplits = 32;     // split-K partitions of one request's KV range

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

__device__ __forceinline__ uint16_t f32_to_bf16_bits(float f) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

// x = hi + lo + O(2^-17 |x|): the two-term bf16 split that lets fp32 activations go through the
// bf16 tensor-core path without being rounded to 8 bits of mantissa.
__device__ __forceinline__ void split_bf16(float x, uint16_t& hi, uint16_t& lo) {
    __nv_bfloat16 h = __float2bfloat16_rn(x);
    hi = __bfloat16_as_ushort(h);
    lo = __bfloat16_as_ushort(__float2bfloat16_rn(x - __bfloat162float(h)));
}

__device__ __forceinline__ uint32_t pack2(uint16_t a, uint16_t b) { return (uint32_t)a | ((uint32_t)b << 16); }

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint4& a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---- shared-memory barriers, bulk asynchronous copies, programmatic dependent launch ----------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// Orders this thread's (and, after a barrier, the CTA's) ordinary shared-memory accesses before later writes of the
// copy engine to the same shared memory.
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Wait for the barrier phase with the given parity.  Bounded: gives up (returns false) after about two
// seconds so that a protocol error can never hang the GPU; callers then raise the kernel's error word.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((it & 1023u) == 1023u) {
            const uint64_t now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > 2000000000ull) return false;
        }
    }
}
// Contiguous global -> shared copy by the copy engine; completion is counted in bytes on `bar`.
// Both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// Weights are read once per pass: their lines are marked evict-first in L2, so that the 400 MB a layer streams
// do not push out the few megabytes every phase boundary depends on (residual stream, activations, partial sums,
// rotary tables), which would otherwise come back from HBM behind the weight stream's own queue.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar), "l"(pol)
                 : "memory");
}
// Hint: pull a contiguous global range into L2 (no destination, no completion to wait for).  Address 16-byte
// aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
// What a kernel pulls into L2 on behalf of its successor while its own demand on HBM ebbs (its tail: split-K
// reduction, epilogue, grid hand-over leave HBM idle for several microseconds).  The successor's weights are cut
// into `runs` contiguous ranges of `run_bytes` (one per successor CTA); the successor copies the first `skip`
// bytes of its range into shared memory by itself before its dependency wait, so the hint covers the `len`
// bytes after those.  Purely a hint: results never depend on it.
struct L2Prefetch {
    const unsigned char* ptr;   // null: nothing to prefetch
    uint32_t run_bytes, skip, len;
    int runs;
};
// CTA `cta` of `n_ctas` issues the hints of runs cta, cta + n_ctas, ...: `n_thr` threads call this with their index
// `tid`, one 128-byte line per thread and step, through the load/store path (the copy engine's queue stays free for
// the successor's own copies).
__device__ __forceinline__ void l2_prefetch_issue(const L2Prefetch& pf, int cta, int n_ctas, int tid, int n_thr) {
    if (pf.ptr == nullptr) return;
    for (int r = cta; r < pf.runs; r += n_ctas) {
        const unsigned char* p = pf.ptr + (size_t)r * pf.run_bytes + pf.skip;
        for (uint32_t o = (uint32_t)tid * 128u; o < pf.len; o += (uint32_t)n_thr * 128u)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p + o) : "memory");
    }
}
// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may start
// while its predecessor drains; pdl_wait() blocks until the predecessor has completed and its writes
// are visible, pdl_launch_dependents() lets the successor start early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                     Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// The same with a thread-block cluster of `cluster_x` consecutive CTAs along x (1: no cluster).
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                             cudaStream_t st, int cluster_x, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    int n = 1;
    if (cluster_x > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)cluster_x;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        n = 2;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- split-bf16 activation arrays ("xf"): B fragments of mma.m16n8k16 in global memory ----------
// Layout [token block][k16 step][n8 tile][lane] of uint4 = {hi.b0, hi.b1, lo.b0, lo.b1} where, for lane
// = 4*g + t, b0 holds k = 2t, 2t+1 and b1 holds k = 2t+8, 2t+9 of token 8*tile + g.
// Stores the pair (k, k+1), k even, of one token.  KS = K/16, NT = tiles per token block.
__device__ __forceinline__ void xf_store_pair(uint32_t* xf, int tok, int k, float v0, float v1, int KS, int NT) {
    const int tb = tok / (8 * NT), nt = (tok >> 3) % NT, g = tok & 7;
    const int ks = k >> 4, kk = k & 15, t = (kk & 7) >> 1, half = kk >> 3;
    const size_t slot = ((size_t)(tb * KS + ks) * NT + nt) * 32 + g * 4 + t;
    uint16_t h0, l0, h1, l1;
    split_bf16(v0, h0, l0);
    split_bf16(v1, h1, l1);
    xf[slot * 4 + half] = pack2(h0, h1);
    xf[slot * 4 + 2 + half] = pack2(l0, l1);
}

// 16-bit variant: stores one element (its hi and lo halves) of an xf array.
__device__ __forceinline__ void xf_store_one(uint16_t* xf, int tok, int k, float v, int KS, int NT) {
    const int tb = tok / (8 * NT), nt = (tok >> 3) % NT, g = tok & 7;
    const int ks = k >> 4, kk = k & 15, t = (kk & 7) >> 1, half = kk >> 3;
    const size_t slot = ((size_t)(tb * KS + ks) * NT + nt) * 32 + g * 4 + t;
    uint16_t h, l;
    split_bf16(v, h, l);
    xf[slot * 8 + half * 2 + (kk & 1)] = h;
    xf[slot * 8 + 4 + half * 2 + (kk & 1)] = l;
}

// ---- "xd" activation arrays: the K-major B operand of tcgen05.mma (the dense GEMM's input), in global memory ----
// Token blocks of `tbs` tokens (a multiple of 16).  Per (token block, k16 step): the bf16 hi tile then the lo tile,
// tbs * 32 bytes each, cut into 8x8 core matrices: element (token t, k) of a tile at
// ((t / 8) * 2 + (k / 8) % 2) * 128 + (t % 8) * 16 + (k % 8) * 2.
__device__ __forceinline__ void xd_store_one(uint16_t* xd, int tok, int k, float v, int KS, int tbs) {
    const int tb = tok / tbs, tl = tok % tbs;
    uint16_t h, l;
    split_bf16(v, h, l);
    unsigned char* b = reinterpret_cast<unsigned char*>(xd) + ((size_t)tb * KS + (k >> 4)) * (size_t)(tbs * 64) +
                       (((tl >> 3) * 2 + ((k >> 3) & 1)) * 128 + (tl & 7) * 16 + (k & 7) * 2);
    *reinterpret_cast<uint16_t*>(b) = h;
    *reinterpret_cast<uint16_t*>(b + tbs * 32) = l;
}
// In either layout an element's index (in 16-bit units) is the sum of a part fixed by its token and the first k16 step
// ks0 of a block of columns, and a part fixed by the column's offset dk inside that block; the lo half follows the hi
// half at a fixed distance.  Epilogues that walk tokens x columns compute each part once instead of dividing per element.
__device__ __forceinline__ uint32_t act_index_row(int tok, int ks0, int KS, int NT, int tbs) {
    if (tbs > 0) {
        const int tb = tok / tbs, tl = tok % tbs;
        return (uint32_t)(((tb * KS + ks0) * (tbs * 64) + (tl >> 3) * 256 + (tl & 7) * 16) >> 1);
    }
    const int tb = tok / (8 * NT), nt = (tok >> 3) % NT, g = tok & 7;
    return (uint32_t)((((tb * KS + ks0) * NT + nt) * 32 + g * 4) * 8);
}
__device__ __forceinline__ uint32_t act_index_col(int dk, int NT, int tbs) {
    const int kk = dk & 15;
    if (tbs > 0) return (uint32_t)(((dk >> 4) * (tbs * 64) + (kk >> 3) * 128 + (kk & 7) * 2) >> 1);
    return (uint32_t)((dk >> 4) * NT * 256 + ((kk & 7) >> 1) * 8 + (kk >> 3) * 2 + (kk & 1));
}
__device__ __forceinline__ uint32_t act_index_lo(int tbs) { return tbs > 0 ? (uint32_t)tbs * 16u : 4u; }
__device__ __forceinline__ void act_store_at(uint16_t* dst, uint32_t idx, uint32_t lo, float v) {
    uint16_t h, l;
    split_bf16(v, h, l);
    dst[idx] = h;
    dst[idx + lo] = l;
}
// Store one activation in whichever layout its consumer reads: tbs > 0: an xd array with that block size; tbs == 0:
// the small-M kernel's fragment order with NT token tiles per block.
__device__ __forceinline__ void act_store_one(uint16_t* dst, int tok, int k, float v, int KS, int NT, int tbs) {
    if (tbs > 0) xd_store_one(dst, tok, k, v, KS, tbs);
    else xf_store_one(dst, tok, k, v, KS, NT);
}

// ---- thread-block clusters: barrier and distributed shared memory --------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctaid_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctaid.x;" : "=r"(r));
    return r;
}
// Every thread of every CTA of the cluster must execute this (hardware barrier, release/acquire).
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local_smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float dsmem_ld_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void dsmem_st_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// Per-pass metadata that lives in device memory (uploaded once per call).
struct PassMeta {
    const int32_t* row_item;   // [M] batch item of each row
    const int32_t* row_pos;    // [M] absolute position of each row in its request
    const int32_t* row_tok;    // [M] token id of each row
    const int32_t* it_slot;    // [n_items] request slot (row of the block table)
    const int32_t* it_row0;    // [n_items] first row of the item
    const int32_t* it_rows;    // [n_items] rows of the item (k+1)
    const int32_t* it_base;    // [n_items] cached positions before this pass
    const int32_t* it_nsplit;  // [n_items] key splits
    const int32_t* it_chunk;   // [n_items] keys per split (multiple of the page size)
    const int32_t* it_part0;   // [n_items] first slot of the item in the attention partial arrays
    const int32_t* it_order;   // [n_items] items by decreasing number of keys: the order their attention CTAs launch in
    const int32_t* block_tab;  // [max_requests][max_pages] page ids, indexed by request slot
    int max_pages;
};

// Offset (in elements) of K (kv=0) or V (kv=1) element (slot, e) of a head inside the paged pool:
// layout [layer][page][kv][head][slot/8][e/8][slot%8][e%8].  Inside a (page, head) block the rows sit in groups of
// eight, cut into 8-element (16-byte) pieces, the eight rows' pieces of the same columns next to each other: 128
// contiguous bytes are an 8 x 8 "core matrix" of the tensor cores' shared-memory operands, so a page copied to
// shared memory as it is serves as the K-major operand of Q K^T (rows = keys) and as the MN-major operand of P V
// (rows = head dimensions) alike.  The page size is a multiple of 8.
__device__ __host__ __forceinline__ size_t kv_row_offset(int slot, int hd) {          // of element 0 of a row inside its block
    return (size_t)(slot >> 3) * hd * 8 + (size_t)(slot & 7) * 8;
}
__device__ __host__ __forceinline__ size_t kv_col_offset(int e) { return (size_t)(e >> 3) * 64 + (size_t)(e & 7); }
__device__ __host__ __forceinline__ size_t kv_index(int layer, int n_pages, int page, int kv, int n_kv_heads,
                                                    int head, int page_size, int slot, int hd, int e) {
    return ((((size_t)layer * n_pages + page) * 2 + kv) * n_kv_heads + head) * page_size * (size_t)hd +
           kv_row_offset(slot, hd) + kv_col_offset(e);
}

}  // namespace pipesd
