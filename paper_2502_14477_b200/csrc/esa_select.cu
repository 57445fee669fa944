// Eq. 8 + Eq. 2: proximity max-pooling of the aggregated scores and top-k selection.
//
//   s'_j = max_{w = max(j-eps, first)}^{min(j+eps, last)} s_w        (Eq. 8, window clipped to M)
//   M_k  = the k tokens of M with the largest s'                      (Eq. 2)
//
// Ties are the rule, not the exception (each query's arg-max scores exactly 0 and the
// pooling copies every peak to 2*eps+1 neighbours), so the order is total: larger score
// first, lower index first among equal scores.  Scores are handled as order-preserving
// uint32 keys.  One thread-block cluster (8 CTAs, or 16 for small batches) works on one sequence: every CTA pools its
// slice of M, then three radix passes (11 + 11 + 10 bits, each digit's histogram all-reduced
// into every CTA through distributed shared memory) find the k-th largest key T, and an index-ordered
// compaction emits every key > T plus the first (k - #greater) keys == T, which is
// exactly "lowest index wins" and leaves the output ascending.
#include <cooperative_groups.h>

#include "esa_internal.h"

namespace cg = cooperative_groups;

namespace esa {

constexpr int SEL_CLUSTER_MAX = 16;   // CTAs working on one sequence: 8, or 16 (beyond the portable size) for small batches
constexpr int SEL_THREADS = 1024;
constexpr int SEL_BINS = 2048;
constexpr size_t kSelMinDynSmem = 100 * 1024;   // with the static 33 KB: more than half an SM's shared memory
static_assert(SEL_CLUSTER_MAX <= 32, "one lane per lower-ranked CTA in the compaction");

struct SelectParams {
    const uint32_t* skey;   // aggregated keys (unused when pooled != 0)
    const uint32_t* rkey;   // [B * l_C] (pooled mode reads r of query 0)
    uint32_t* pkey;         // pooled keys: out, or in when pooled != 0
    const uint32_t* ghist0; // [B, SEL_BINS] first-digit histograms of pkey (pooled mode)
    int32_t* idx_out;       // [B, top_k]
    int32_t* n_sel_out;     // [B]
    int64_t max_tokens;
    int top_k;
    int eps;
    int pooled;             // the scoring kernel already pooled (keys of P = pooled raw scores) and took the first histogram
    int l_C;
    int slice_cap;          // keys of a CTA's slice that fit in its dynamic shared memory (0: none)
    SeqMeta meta;
};


// Histogram update aggregated over the warp: pooled scores crowd into a handful of bins
// (same sign and exponent), so lanes with equal bins elect one leader that adds their count.
// Must be called by converged lanes named in `active`.
__device__ __forceinline__ void hist_add(uint32_t* hist, uint32_t bin, uint32_t active) {
    const uint32_t peers = __match_any_sync(active, bin);
    if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
}

// Finds, in the cluster-wide histogram `g` of one digit (nb bins, larger bin = larger key),
// the bin holding the krem-th largest remaining key.  Every CTA runs this on its own copy
// and gets the same answer.  Returns through sh_out[0] (bin) and sh_out[1] (keys still to
// place inside that bin).
__device__ __forceinline__ void find_bin(const uint32_t* g, int nb, uint32_t krem, uint32_t* scan_tmp,
                                         uint32_t* sh_out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // each thread owns `per` consecutive bins, highest bins first
    const int per = (nb + SEL_THREADS - 1) / SEL_THREADS;
    uint32_t mine = 0;
    for (int j = 0; j < per; ++j) {
        int bin = nb - 1 - (tid * per + j);
        if (bin >= 0) mine += g[bin];
    }
    uint32_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    if (lane == 31) scan_tmp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = scan_tmp[lane];
        uint32_t wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t n = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += n;
        }
        scan_tmp[lane] = wi - w;   // exclusive warp offsets
    }
    __syncthreads();
    const uint32_t before = scan_tmp[warp] + incl - mine;   // keys in bins above this thread's bins
    if (before < krem && before + mine >= krem) {
        uint32_t acc = before;
        for (int j = 0; j < per; ++j) {
            int bin = nb - 1 - (tid * per + j);
            if (bin < 0) break;
            uint32_t c = g[bin];
            if (acc + c >= krem) {
                sh_out[0] = (uint32_t)bin;
                sh_out[1] = krem - acc;
                break;
            }
            acc += c;
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(SEL_THREADS)
select_topk_kernel(SelectParams p) {
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int n_ctas = (int)gridDim.x;          // = cluster size: one cluster per sequence
    const int b = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    extern __shared__ uint32_t slice_keys[];   // pooled keys of this CTA's slice (when they fit)
    __shared__ uint32_t hist[SEL_BINS];        // this CTA's histogram of the current digit
    __shared__ uint32_t ghist[3][SEL_BINS];    // cluster-wide histograms, one per digit, same in every CTA
    __shared__ uint32_t warp_cnt[2][32];
    __shared__ uint32_t cta_cnt[2];            // (#greater, #equal) in this CTA's slice
    __shared__ uint32_t sh_found[2];
    __shared__ uint32_t scan_tmp[SEL_THREADS / 32];

    const int i_end = p.meta.i_end[b];
    const int l_M = p.meta.m_end[b] - i_end;
    const int k = p.top_k;
    // sequences whose middle part fits in k are emitted whole by another kernel
    // (uniform over the cluster, so no barrier is left waiting)
    if (l_M <= k) return;

    const uint32_t* src = p.skey + (int64_t)b * p.max_tokens;
    uint32_t* pk = p.pkey + (int64_t)b * p.max_tokens;
    const int pooled = p.pooled;

    // slice of this CTA: whole 32-element rows, contiguous
    const int rows32 = (l_M + 31) / 32;
    const int rows_per_cta = (rows32 + n_ctas - 1) / n_ctas;
    const int lo = min(l_M, rank * rows_per_cta * 32);
    const int hi = min(l_M, (rank + 1) * rows_per_cta * 32);

    for (int i = tid; i < SEL_BINS; i += SEL_THREADS) {
        hist[i] = 0;
        ghist[0][i] = ghist[1][i] = ghist[2][i] = 0;
    }
    cluster.sync();     // every CTA's histograms are zero before anyone adds to them remotely
    pdl_wait();         // the scores come from the preceding kernel
    pdl_launch_dependents();
    const float r0 = pooled ? key_to_f32(p.rkey[(int64_t)b * p.l_C]) : 0.f;

    // ---- digit 0: pool (Eq. 8), store pooled keys, histogram of bits 31..21
    // A warp loads 32 consecutive keys starting eps before its first output and slides the
    // window with shuffles: lane i ends with max(key[i .. i+2*eps]) = s' of token first+i, so
    // each key is loaded and converted once; 32 - 2*eps outputs per step.  Positions outside
    // M contribute key 0, which is below every real key (the window is clipped to M).
    // Later passes re-read the slice: from shared memory when it fits, else from pkey (L2).
    const bool in_smem = (hi - lo) <= p.slice_cap;
    const uint32_t* keys = in_smem ? slice_keys : pk + lo;     // keys[i] = s' of token lo + i
    if (pooled) {
        // the scoring kernel left the pooled keys and their first-digit histogram: fetch this CTA's slice
        // (four independent loads per thread and round) and every CTA's copy of the histogram
        if (in_smem) {
            for (int i0 = 0; i0 < hi - lo; i0 += 4 * SEL_THREADS) {
                uint32_t v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * SEL_THREADS + tid;
                    v[u] = (i < hi - lo) ? __ldcg(pk + lo + i) : 0u;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * SEL_THREADS + tid;
                    if (i < hi - lo) slice_keys[i] = v[u];
                }
            }
        }
        for (int i = tid; i < SEL_BINS; i += SEL_THREADS) ghist[0][i] = __ldcg(p.ghist0 + (int64_t)b * SEL_BINS + i);
    } else {
        const int eps = p.eps;
        const int outs = 32 - 2 * eps;
        constexpr int UN = 4;                                   // independent loads in flight per lane
        const int step = (SEL_THREADS / 32) * outs;
        for (int first0 = lo + warp * outs; first0 < hi; first0 += UN * step) {
            uint32_t key[UN];
#pragma unroll
            for (int u = 0; u < UN; ++u) {
                const int mload = first0 + u * step - eps + lane;
                key[u] = (first0 + u * step < hi && mload >= 0 && mload < l_M) ? src[mload] : 0u;
            }
#pragma unroll
            for (int u = 0; u < UN; ++u) {
                const int first = first0 + u * step;
                if (first >= hi) break;                         // uniform over the warp
                uint32_t best = key[u];
                for (int o = 1; o <= 2 * eps; ++o) best = max(best, __shfl_down_sync(0xffffffffu, key[u], o));
                const int m = first + lane;
                const bool valid = lane < outs && m < hi;
                const uint32_t active = __ballot_sync(0xffffffffu, valid);
                if (valid) {
                    pk[m] = best;
                    if (in_smem) slice_keys[m - lo] = best;
                    hist_add(hist, best >> 21, active);
                }
            }
        }
    }

    uint32_t prefix = 0, krem = (uint32_t)k;
    const int shifts[3] = {21, 10, 0};
    const int nbits[3] = {11, 11, 10};
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        __syncthreads();
        // all-reduce of the digit histogram: every non-empty local bin is added to every CTA's copy
        const int nb = 1 << nbits[pass];
        if (!(pooled && pass == 0)) {      // (pooled: the first digit's histogram came complete from global memory)
            for (int i = tid; i < nb; i += SEL_THREADS) {
                const uint32_t c = hist[i];
                if (c) {
                    for (int r = 0; r < n_ctas; ++r) atomicAdd(cluster.map_shared_rank(&ghist[pass][i], r), c);
                }
            }
            cluster.sync();
        }
        find_bin(ghist[pass], nb, krem, scan_tmp, sh_found);
        prefix |= sh_found[0] << shifts[pass];
        krem = sh_found[1];
        if (pass == 2) break;
        // ---- next digit among the keys that match the prefix found so far
        for (int i = tid; i < SEL_BINS; i += SEL_THREADS) hist[i] = 0;
        __syncthreads();
        const int sh = shifts[pass + 1];
        const uint32_t dmask = (1u << nbits[pass + 1]) - 1u;
        const int psh = shifts[pass];          // bits psh and above are fixed
        for (int m0 = lo + warp * 32; m0 < hi; m0 += SEL_THREADS) {
            const int m = m0 + lane;
            const uint32_t key = (m < hi) ? keys[m - lo] : 0u;
            const bool take = (m < hi) && (key >> psh) == (prefix >> psh);
            const uint32_t active = __ballot_sync(0xffffffffu, take);
            if (take) hist_add(hist, (key >> sh) & dmask, active);
        }
    }
    // k-th largest key.  Pooled mode: the keys so far are those of P (raw pooled scores); Eq. 4's
    // s' = fl(P - r) is a monotone map of P, so its k-th largest value is the image of the k-th
    // largest P, and the compaction below runs on the mapped keys (ties of s' included).
    const uint32_t T = pooled ? f32_to_key(key_to_f32(prefix) - r0) : prefix;
    auto final_key = [&](uint32_t key) { return pooled ? f32_to_key(key_to_f32(key) - r0) : key; };

    // ---- ordered compaction
    // each warp owns a contiguous run of 32-element rows of the CTA's slice
    const int cta_rows = (hi - lo + 31) / 32;
    const int rows_per_warp = (cta_rows + 31) / 32;
    const int w_lo = min(hi, lo + warp * rows_per_warp * 32);
    const int w_hi = min(hi, lo + (warp + 1) * rows_per_warp * 32);
    uint32_t n_gt = 0, n_eq = 0;
    for (int m = w_lo + lane; m < w_hi; m += 32) {
        uint32_t key = final_key(keys[m - lo]);
        n_gt += key > T;
        n_eq += key == T;
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        n_gt += __shfl_xor_sync(0xffffffffu, n_gt, o);
        n_eq += __shfl_xor_sync(0xffffffffu, n_eq, o);
    }
    if (lane == 0) {
        warp_cnt[0][warp] = n_gt;
        warp_cnt[1][warp] = n_eq;
    }
    __syncthreads();
    if (warp == 0) {
        uint32_t g = warp_cnt[0][lane], e = warp_cnt[1][lane];
        uint32_t gi = g, ei = e;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t a = __shfl_up_sync(0xffffffffu, gi, o);
            uint32_t c = __shfl_up_sync(0xffffffffu, ei, o);
            if (lane >= o) { gi += a; ei += c; }
        }
        warp_cnt[0][lane] = gi - g;     // exclusive offsets inside the CTA
        warp_cnt[1][lane] = ei - e;
        if (lane == 31) { cta_cnt[0] = gi; cta_cnt[1] = ei; }
    }
    cluster.sync();
    // counts of the lower-ranked CTAs: one remote read per lane, all in flight together
    uint32_t gt_before = 0, eq_before = 0, gt_all = 0;
    if (lane < n_ctas) {
        gt_all = *cluster.map_shared_rank(&cta_cnt[0], lane);
        if (lane < rank) {
            gt_before = gt_all;
            eq_before = *cluster.map_shared_rank(&cta_cnt[1], lane);
        }
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        gt_before += __shfl_xor_sync(0xffffffffu, gt_before, o);
        eq_before += __shfl_xor_sync(0xffffffffu, eq_before, o);
        gt_all += __shfl_xor_sync(0xffffffffu, gt_all, o);
    }
    krem = (uint32_t)k - gt_all;      // keys equal to T still to take (= the radix passes' remainder; recounted for the mapped keys)
    gt_before += warp_cnt[0][warp];
    eq_before += warp_cnt[1][warp];
    int32_t* out = p.idx_out + (int64_t)b * p.top_k;
    for (int m0 = w_lo; m0 < w_hi; m0 += 32) {
        int m = m0 + lane;
        uint32_t key = (m < w_hi) ? final_key(keys[m - lo]) : 0u;
        bool gt = (m < w_hi) && key > T;
        bool eq = (m < w_hi) && key == T;
        uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
        uint32_t lt_mask = (1u << lane) - 1u;
        uint32_t my_gt = gt_before + __popc(bg & lt_mask);
        uint32_t my_eq = eq_before + __popc(be & lt_mask);
        if (gt || (eq && my_eq < krem)) {
            uint32_t pos = my_gt + min(my_eq, krem);
            if (pos < (uint32_t)k) out[pos] = i_end + m;
        }
        gt_before += __popc(bg);
        eq_before += __popc(be);
    }
    if (rank == 0 && tid == 0) p.n_sel_out[b] = k;
    cluster.sync();   // keep every CTA's shared memory alive until remote reads are done
}

// Sequences whose middle part is not larger than k: every middle token is selected.
__global__ void select_all_kernel(int32_t* idx_out, int32_t* n_sel_out, int top_k, int only_small,
                                  SeqMeta meta) {
    const int b = blockIdx.y;
    const int i_end = meta.i_end[b];
    const int l_M = meta.m_end[b] - i_end;
    if (only_small && l_M > top_k) return;
    const int n = min(l_M, top_k);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
        idx_out[(int64_t)b * top_k + i] = i_end + i;
    if (blockIdx.x == 0 && threadIdx.x == 0) n_sel_out[b] = n;
}

// r: key of the row maximum to subtract (decode: pkey holds the pooled raw scores), or null
__global__ void read_pooled_kernel(const uint32_t* __restrict__ pkey, const uint32_t* __restrict__ r,
                                   float* __restrict__ dst, int64_t n) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = r ? key_to_f32(pkey[i]) - key_to_f32(*r) : key_to_f32(pkey[i]);
}

cudaError_t launch_select(esa_ctx* ctx, int B, int l_C, const SeqMeta& meta, int max_lM, int32_t* idx_out,
                          int32_t* n_sel_out, cudaStream_t st) {
    SelectParams p;
    p.skey = ctx->skey; p.rkey = ctx->rkey; p.pkey = ctx->pkey;
    p.idx_out = idx_out; p.n_sel_out = n_sel_out;
    p.max_tokens = ctx->cfg.max_tokens; p.top_k = ctx->cfg.top_k; p.eps = ctx->cfg.eps;
    p.pooled = (l_C == 1) ? 1 : 0; p.ghist0 = ctx->ghist0; p.l_C = l_C; p.meta = meta;
    cudaError_t e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    // 16 CTAs per sequence while the whole batch still fits half the machine and the device can
    // place such a cluster; 10 for somewhat larger batches; else the portable 8
    static int can16 = -1;
    if (can16 < 0) {
        cudaLaunchConfig_t probe = {};
        probe.gridDim = dim3(SEL_CLUSTER_MAX, 1);
        probe.blockDim = dim3(SEL_THREADS);
        probe.dynamicSmemBytes = kSelMinDynSmem;
        cudaLaunchAttribute pa[1];
        pa[0].id = cudaLaunchAttributeClusterDimension;
        pa[0].val.clusterDim.x = SEL_CLUSTER_MAX;
        pa[0].val.clusterDim.y = 1;
        pa[0].val.clusterDim.z = 1;
        probe.attrs = pa;
        probe.numAttrs = 1;
        int n = 0;
        can16 = (cudaOccupancyMaxActiveClusters(&n, select_topk_kernel, &probe) == cudaSuccess && n > 0) ? 1 : 0;
        if (!can16) cudaGetLastError();
    }
    // (measured on 148 SMs with 8 sequences: clusters of 10 beat 8 by a few percent, clusters of 12 or 16 place badly)
    int n_ctas = 8;
    if (can16 && B * SEL_CLUSTER_MAX <= ctx->num_sms / 2) n_ctas = SEL_CLUSTER_MAX;
    else if (can16 && B * 10 * 5 <= ctx->num_sms * 3) n_ctas = 10;
    // dynamic shared memory for a CTA's slice of pooled keys (largest sequence of the call)
    const int rows32 = (max_lM + 31) / 32;
    const int slice = ((rows32 + n_ctas - 1) / n_ctas) * 32;
    size_t smem = (size_t)slice * 4;
    if (smem > 160 * 1024) smem = 0;
    p.slice_cap = (int)(smem / 4);
    // One CTA per SM: the passes are bound by instruction issue, and two of these 1024-thread CTAs on
    // one SM (their registers and small slices would allow it) run at half speed each while other SMs
    // idle -- measured: the block scheduler does pack them.
    if (smem < kSelMinDynSmem) smem = kSelMinDynSmem;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_ctas, B);
    cfg.blockDim = dim3(SEL_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = n_ctas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    e = cudaLaunchKernelEx(&cfg, select_topk_kernel, p);
    if (e != cudaSuccess) return e;
    ctx->launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_select_all(esa_ctx* ctx, int B, const SeqMeta& meta, int32_t* idx_out,
                              int32_t* n_sel_out, cudaStream_t st) {
    int gx = (ctx->cfg.top_k + 255) / 256;
    if (gx > 64) gx = 64;
    if (gx < 1) gx = 1;
    select_all_kernel<<<dim3(gx, B), 256, 0, st>>>(idx_out, n_sel_out, ctx->cfg.top_k, 1, meta);
    ctx->launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_read_pooled(esa_ctx* ctx, int b, float* dst_dev, int64_t n, cudaStream_t st) {
    read_pooled_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(ctx->pkey + (int64_t)b * ctx->cfg.max_tokens,
                                                                   ctx->last_decode ? ctx->rkey + b : nullptr, dst_dev, n);
    ctx->launches += 1;
    return cudaGetLastError();
}

}  // namespace esa
