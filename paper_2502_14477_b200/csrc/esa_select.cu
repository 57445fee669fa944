// Eq. 8 + Eq. 2: proximity max-pooling of the aggregated scores and top-k selection.
//
//   s'_j = max_{w = max(j-eps, first)}^{min(j+eps, last)} s_w        (Eq. 8, window clipped to M)
//   M_k  = the k tokens of M with the largest s'                      (Eq. 2)
//
// Ties are the rule, not the exception (each query's arg-max scores exactly 0 and the
// pooling copies every peak to 2*eps+1 neighbours), so the order is total: larger score
// first, lower index first among equal scores.  Scores are handled as order-preserving
// uint32 keys.
//
// The selection kernel starts from the pooled keys and the histogram of their top 11 bits
// (both left by the scoring kernels, or by pool_hist_kernel below for the scoring paths that
// do not pool).  It runs in two phases inside one launch, and no CTA ever waits for another:
//   1. every CTA owns a slice of 8192 consecutive tokens.  From the histogram it finds the bin
//      b0 that holds the k-th largest key, and copies the keys that can still matter -- those
//      not below the lower edge of b0 -- with their positions, in index order, to its slice of
//      a candidate list; then it draws an arrival ticket.
//      Along the way the CTAs add up, for the whole sequence, the histogram of the next 11 bits
//      among the keys of bin b0.
//   2. the CTA that draws the last ticket of a sequence gathers the candidate lists (a few
//      thousand entries, shared memory).  The second digit of the k-th largest key T comes from
//      that histogram; the few keys that share T's top 22 bits are ranked directly (a histogram
//      pass over the last 10 bits if they are many: long runs of equal scores).  Then every
//      candidate with key > T plus the first (k - #greater) candidates with key == T in index
//      order are emitted: exactly "lowest index wins", and the output is ascending.
// With one query per sequence (decode) the scoring kernel pooled the raw scores P; Eq. 4's
// s' = fl(P - r) is a monotone map of P.  T is found among the P keys as above; phase 1 keeps the
// keys whose image is not below the image of b0's lower edge (a superset of what can matter, and
// at least k of them), and the final comparison against T's image runs on the mapped keys: exactly
// the selection on s', ties (distinct P with equal images included) broken by index.
#include "esa_internal.h"

namespace esa {

constexpr int SEL_THREADS = 1024;
constexpr int SEL_SLICE = 8192;       // tokens per CTA in phase 1
constexpr int SEL_PER = SEL_SLICE / SEL_THREADS;
constexpr int SEL_ROWS = SEL_SLICE / 32;
constexpr int SEL_BINS = 2048;
constexpr int SEL_STAGE_CAP = 12288;  // candidates the last CTA can stage in shared memory (keys and positions)
constexpr int SEL_MAX_SLICES_SMEM = 1024;
constexpr int SEL_LIST_CAP = 256;     // keys sharing the threshold's top 22 bits that are ranked directly (more: a histogram pass)

struct SelectParams {
    const uint32_t* pkey;   // [B, max_tokens] pooled keys (mapped != 0: of the pooled raw scores P)
    const uint32_t* ghist0; // [B, SEL_BINS] histogram of pkey's top 11 bits
    uint32_t* ghist1;       // [B, SEL_BINS] histogram of the next 11 bits among the keys of bin b0; 0 between launches
    const uint32_t* rkey;   // [B * l_C] (mapped mode reads r of query 0)
    uint32_t* ckey;         // [B, max_tokens] candidate keys, slice s at s * SEL_SLICE
    int32_t* cidx;          // [B, max_tokens] candidate positions (absolute), same layout
    int* slice_cnt;         // [B, slice_stride] candidates per slice
    int* ticket;            // [B] arrivals; 0 between launches
    int32_t* idx_out;       // [B, top_k]
    int32_t* n_sel_out;     // [B]
    int64_t max_tokens;
    int slice_stride;
    int top_k;
    int mapped;
    int l_C;
    SeqMeta meta;
};

// Histogram update aggregated over the warp: pooled scores crowd into a handful of bins
// (same sign and exponent), so lanes with equal bins elect one leader that adds their count.
// Must be called by converged lanes named in `active`.
__device__ __forceinline__ void hist_add(uint32_t* hist, uint32_t bin, uint32_t active) {
    const uint32_t peers = __match_any_sync(active, bin);
    if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
}

// Finds, in the histogram `g` of one digit (nb <= SEL_BINS bins, larger bin = larger key), the bin
// holding the krem-th largest remaining key.  Returns through sh_out[0] (bin) and sh_out[1] (keys
// still to place inside that bin).  Whole CTA; ends with a barrier.
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
        uint32_t w = lane < SEL_THREADS / 32 ? scan_tmp[lane] : 0u;
        uint32_t wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t n = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += n;
        }
        if (lane < SEL_THREADS / 32) scan_tmp[lane] = wi - w;   // exclusive warp offsets
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

// Exclusive scan of one value per warp-row through shared memory: cnt[0 .. n) -> offsets in place,
// total returned to every thread.  n <= SEL_THREADS.  Whole CTA.
__device__ __forceinline__ int block_exclusive_scan(int* cnt, int n, int* warp_tot) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int v = tid < n ? cnt[tid] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int x = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += x;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < SEL_THREADS / 32 ? warp_tot[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int x = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += x;
        }
        if (lane < SEL_THREADS / 32) warp_tot[lane] = wi - w;
        if (lane == 31) warp_tot[32] = wi;
    }
    __syncthreads();
    if (tid < n) cnt[tid] = warp_tot[warp] + incl - v;
    const int total = warp_tot[32];
    __syncthreads();
    return total;
}

__global__ void __launch_bounds__(SEL_THREADS)
select_topk_kernel(SelectParams p) {
    const int b = blockIdx.y;
    const int slice = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    extern __shared__ uint32_t sel_dyn[];          // last CTA: slice offsets, then the staged candidate keys and positions
    __shared__ uint32_t hist[SEL_BINS];
    __shared__ int row_cnt[SEL_THREADS];           // phase 1: candidates per 32-token row; phase 2: slice offsets (first part)
    __shared__ int warp_tot[33];
    __shared__ uint32_t scan_tmp[SEL_THREADS / 32];
    __shared__ uint32_t sh_found[2];
    __shared__ uint32_t lst[SEL_LIST_CAP];         // last CTA: the keys that share the threshold's top 22 bits
    __shared__ uint32_t lst_n;
    __shared__ uint32_t warp_cnt[2][SEL_THREADS / 32];
    __shared__ int sh_last;

    const int i_end = p.meta.i_end[b];
    const int l_M = p.meta.m_end[b] - i_end;
    const int k = p.top_k;
    // sequences whose middle part fits in k are emitted whole by another kernel
    if (l_M <= k) return;
    const int n_slices = (l_M + SEL_SLICE - 1) / SEL_SLICE;
    if (slice >= n_slices) return;

    pdl_wait();         // the keys and the histogram come from the preceding kernel
    pdl_launch_dependents();
    const int mapped = p.mapped;
    const float r0 = mapped ? key_to_f32(p.rkey[(int64_t)b * p.l_C]) : 0.f;
    const uint32_t* pk = p.pkey + (int64_t)b * p.max_tokens;
    uint32_t* ck = p.ckey + (int64_t)b * p.max_tokens;
    int32_t* ci = p.cidx + (int64_t)b * p.max_tokens;

    // ---- phase 1: this slice's keys (in flight while the histogram is scanned)
    const int base = slice * SEL_SLICE;
    uint32_t key[SEL_PER];
#pragma unroll
    for (int j = 0; j < SEL_PER; ++j) {
        const int m = base + j * SEL_THREADS + tid;
        key[j] = m < l_M ? __ldcg(pk + m) : 0u;
    }
    for (int i = tid; i < SEL_BINS; i += SEL_THREADS) hist[i] = __ldcg(p.ghist0 + (int64_t)b * SEL_BINS + i);
    __syncthreads();
    find_bin(hist, SEL_BINS, (uint32_t)k, scan_tmp, sh_found);
    const uint32_t b0 = sh_found[0];
    const uint32_t krem0 = sh_found[1];            // keys of bin b0 among the k largest
    const uint32_t edge = b0 << 21;                // smallest key of bin b0
    const uint32_t cut = mapped ? f32_to_key(key_to_f32(edge) - r0) : edge;
    // (the candidate lists keep the keys as they came; `final_key` is the key the order is decided on)
    auto final_key = [&](uint32_t kv) { return mapped ? f32_to_key(key_to_f32(kv) - r0) : kv; };
    // second radix digit of the keys of bin b0, for the whole sequence: every CTA adds its slice's share
    for (int i = tid; i < SEL_BINS; i += SEL_THREADS) hist[i] = 0u;
    __syncthreads();
    bool cand[SEL_PER];
#pragma unroll
    for (int j = 0; j < SEL_PER; ++j) {
        const int m = base + j * SEL_THREADS + tid;
        cand[j] = m < l_M && final_key(key[j]) >= cut;
        const bool surv = m < l_M && (key[j] >> 21) == b0;
        const uint32_t active = __ballot_sync(0xffffffffu, surv);
        if (surv) hist_add(hist, (key[j] >> 10) & (SEL_BINS - 1), active);
    }
    // candidates in index order: row r = j * 32 + warp holds tokens base + 32 r .. + 31
#pragma unroll
    for (int j = 0; j < SEL_PER; ++j) {
        const uint32_t bal = __ballot_sync(0xffffffffu, cand[j]);
        if (lane == 0) row_cnt[j * (SEL_THREADS / 32) + warp] = __popc(bal);
    }
    __syncthreads();
    for (int i = tid; i < SEL_BINS; i += SEL_THREADS) {
        const uint32_t c = hist[i];
        if (c) atomicAdd(p.ghist1 + (int64_t)b * SEL_BINS + i, c);
    }
    const int n_cand = block_exclusive_scan(row_cnt, SEL_ROWS, warp_tot);
#pragma unroll
    for (int j = 0; j < SEL_PER; ++j) {
        const int m = base + j * SEL_THREADS + tid;
        const bool take = cand[j];
        const uint32_t bal = __ballot_sync(0xffffffffu, take);
        if (take) {
            const int pos = base + row_cnt[j * (SEL_THREADS / 32) + warp] + __popc(bal & ((1u << lane) - 1u));
            ck[pos] = key[j];
            ci[pos] = i_end + m;
        }
    }
    if (tid == 0) p.slice_cnt[(int64_t)b * p.slice_stride + slice] = n_cand;
    __threadfence();                                   // every thread's writes (candidates, histogram, count) before the ticket
    __syncthreads();
    if (tid == 0) {
        const int t = atomicAdd(p.ticket + b, 1);
        sh_last = t == n_slices - 1;
        if (sh_last) p.ticket[b] = 0;              // ready for the next launch
    }
    __syncthreads();
    if (!sh_last) return;
    __threadfence();

    // ---- phase 2 (one CTA per sequence).  The second digit of the k-th largest pooled key T comes from the
    // histogram the CTAs of phase 1 added up (its first digit is b0); it is read first, so that the keys that
    // share those 22 bits can be picked out while the candidates pass through the registers on their way to
    // shared memory.  (The first 32 slice counts are requested at the same time.)
    const int cnt_first = (warp == 0 && lane < n_slices) ? __ldcg(p.slice_cnt + (int64_t)b * p.slice_stride + lane) : 0;
    for (int i = tid; i < SEL_BINS; i += SEL_THREADS) {
        hist[i] = __ldcg(p.ghist1 + (int64_t)b * SEL_BINS + i);
        p.ghist1[(int64_t)b * SEL_BINS + i] = 0u;                     // ready for the next launch
    }
    if (tid == 0) lst_n = 0u;
    __syncthreads();
    find_bin(hist, SEL_BINS, krem0, scan_tmp, sh_found);
    const uint32_t top22 = (b0 << 11) | sh_found[0];
    const uint32_t krem1 = sh_found[1];
    // offsets of the slices' candidate lists:
    // slice counts -> exclusive offsets, SEL_THREADS slices per round (shared memory holds the first
    // SEL_MAX_SLICES_SMEM offsets; longer sequences re-read the counts)
    int* soff = reinterpret_cast<int*>(sel_dyn);   // [n_slices + 1] when it fits, ahead of the staged candidates
    const bool offs_in_smem = n_slices + 1 <= SEL_MAX_SLICES_SMEM;
    if (warp == 0) {
        // one warp scans the slice counts, 32 per round (a sequence has a few dozen slices)
        int run = 0;
        for (int s0 = 0; s0 < n_slices; s0 += 32) {
            const int s = s0 + lane;
            const int c = s0 == 0 ? cnt_first : (s < n_slices ? __ldcg(p.slice_cnt + (int64_t)b * p.slice_stride + s) : 0);
            int incl = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int x = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += x;
            }
            if (offs_in_smem && s < n_slices) soff[s] = run + incl - c;
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            if (offs_in_smem) soff[n_slices] = run;
            warp_tot[32] = run;
        }
    }
    __syncthreads();
    const int total = warp_tot[32];
    const int C = total;                           // >= k candidates in all
    uint32_t* skeys = sel_dyn + SEL_MAX_SLICES_SMEM;
    int32_t* sidx = reinterpret_cast<int32_t*>(skeys + SEL_STAGE_CAP);
    const bool staged = offs_in_smem && C <= SEL_STAGE_CAP;
    const uint32_t* dk;
    const int32_t* di;
    if (staged) {
        // dense copy in shared memory: candidate i of the dense order lives in the slice s with
        // soff[s] <= i < soff[s + 1].  Eight candidates per thread and round, their sixteen loads in flight together.
        auto src_of = [&](int i) {
            int lo = 0, hi = n_slices;                     // invariant: soff[lo] <= i < soff[hi]
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (soff[mid] <= i) lo = mid; else hi = mid;
            }
            return lo * SEL_SLICE + (i - soff[lo]);
        };
        for (int i0 = tid; i0 < C; i0 += 8 * SEL_THREADS) {
            int src[8];
            uint32_t kk[8];
            int32_t ii[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * SEL_THREADS;
                src[u] = i < C ? src_of(i) : 0;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                kk[u] = __ldcg(ck + src[u]);
                ii[u] = __ldcg(ci + src[u]);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * SEL_THREADS;
                if (i < C) {
                    skeys[i] = kk[u];
                    sidx[i] = ii[u];
                    if ((kk[u] >> 10) == top22) {
                        const uint32_t at = atomicAdd(&lst_n, 1u);
                        if (at < SEL_LIST_CAP) lst[at] = kk[u];
                    }
                }
            }
        }
        dk = skeys;
        di = sidx;
    } else {
        // too many candidates (long runs of equal scores): close the gaps in place, slice by slice
        // (a slice's list moves to a lower or equal address; it is read into registers first)
        int off = 0;
        for (int s = 0; s < n_slices; ++s) {
            const int c = __ldcg(p.slice_cnt + (int64_t)b * p.slice_stride + s);
            uint32_t kk[SEL_PER];
            int32_t ii[SEL_PER];
#pragma unroll
            for (int j = 0; j < SEL_PER; ++j) {
                const int e = j * SEL_THREADS + tid;
                kk[j] = e < c ? __ldcg(ck + s * SEL_SLICE + e) : 0u;
                ii[j] = e < c ? __ldcg(ci + s * SEL_SLICE + e) : 0;
            }
            __syncthreads();
#pragma unroll
            for (int j = 0; j < SEL_PER; ++j) {
                const int e = j * SEL_THREADS + tid;
                if (e < c) {
                    ck[off + e] = kk[j];
                    ci[off + e] = ii[j];
                }
            }
            off += c;
            __syncthreads();
        }
        dk = ck;
        di = ci;
    }
    __syncthreads();

    // ---- k-th largest pooled key T: the handful of keys that share its top 22 bits are ranked directly
    if (!staged) {
        for (int i = tid; i < C; i += SEL_THREADS) {
            const uint32_t kv = dk[i];
            if ((kv >> 10) == top22) {
                const uint32_t at = atomicAdd(&lst_n, 1u);
                if (at < SEL_LIST_CAP) lst[at] = kv;
            }
        }
        __syncthreads();
    }
    const uint32_t n_lst = lst_n;
    if (n_lst <= SEL_LIST_CAP) {
        if (tid < (int)n_lst) {
            const uint32_t kv = lst[tid];
            uint32_t g = 0, e = 0;
            for (uint32_t j = 0; j < n_lst; ++j) {
                const uint32_t o = lst[j];
                g += o > kv;
                e += o == kv;
            }
            if (g < krem1 && krem1 <= g + e) sh_found[0] = kv;         // (every key equal to T writes the same value)
        }
        __syncthreads();
    } else {
        // many keys share the 22 bits (long runs of equal scores): one more histogram pass over the last 10 bits
        for (int i = tid; i < SEL_BINS; i += SEL_THREADS) hist[i] = 0;
        __syncthreads();
        for (int i0 = warp * 32; i0 < C; i0 += SEL_THREADS) {
            const int i = i0 + lane;
            const uint32_t kv = i < C ? dk[i] : 0u;
            const bool take = i < C && (kv >> 10) == top22;
            const uint32_t active = __ballot_sync(0xffffffffu, take);
            if (take) hist_add(hist, kv & 1023u, active);
        }
        __syncthreads();
        find_bin(hist, 1024, krem1, scan_tmp, sh_found);
        if (tid == 0) sh_found[0] |= top22 << 10;
        __syncthreads();
    }
    // the order is decided on the final keys: Eq. 4's subtraction is monotone, so the k-th largest final key
    // is the image of the k-th largest pooled key
    const uint32_t T = final_key(sh_found[0]);

    // ---- ordered compaction: each warp owns a contiguous run of 32-candidate rows
    const int rows = (C + 31) / 32;
    const int rows_per_warp = (rows + SEL_THREADS / 32 - 1) / (SEL_THREADS / 32);
    const int w_lo = min(C, warp * rows_per_warp * 32);
    const int w_hi = min(C, (warp + 1) * rows_per_warp * 32);
    uint32_t n_gt = 0, n_eq = 0;
    for (int i = w_lo + lane; i < w_hi; i += 32) {
        const uint32_t kv = final_key(dk[i]);
        n_gt += kv > T;
        n_eq += kv == T;
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
    uint32_t gt_before = 0, eq_before = 0, gt_all = 0;
    {
        const uint32_t g = lane < SEL_THREADS / 32 ? warp_cnt[0][lane] : 0u;
        const uint32_t e = lane < SEL_THREADS / 32 ? warp_cnt[1][lane] : 0u;
        gt_all = g;
        gt_before = lane < warp ? g : 0u;
        eq_before = lane < warp ? e : 0u;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            gt_all += __shfl_xor_sync(0xffffffffu, gt_all, o);
            gt_before += __shfl_xor_sync(0xffffffffu, gt_before, o);
            eq_before += __shfl_xor_sync(0xffffffffu, eq_before, o);
        }
    }
    const uint32_t take_eq = (uint32_t)k - gt_all;      // keys equal to T still to take (= the radix passes' remainder)
    int32_t* out = p.idx_out + (int64_t)b * p.top_k;
    for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
        const int i = i0 + lane;
        const uint32_t kv = i < w_hi ? final_key(dk[i]) : 0u;
        const bool gt = i < w_hi && kv > T;
        const bool eq = i < w_hi && kv == T;
        const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
        const uint32_t lt_mask = (1u << lane) - 1u;
        const uint32_t my_gt = gt_before + __popc(bg & lt_mask);
        const uint32_t my_eq = eq_before + __popc(be & lt_mask);
        if (gt || (eq && my_eq < take_eq)) {
            const uint32_t pos = my_gt + min(my_eq, take_eq);
            if (pos < (uint32_t)k) out[pos] = di[i];
        }
        gt_before += __popc(bg);
        eq_before += __popc(be);
    }
    if (tid == 0) p.n_sel_out[b] = k;
}

// Eq. 8 for the scoring paths that leave unpooled keys: pools skey into pkey and adds the
// histogram of the pooled keys' top 11 bits to ghist0 (zero on entry).  A CTA owns SEL_SLICE
// consecutive tokens and reads eps neighbours on either side; positions outside M contribute
// key 0, which is below every real key (the window is clipped to M).
__global__ void __launch_bounds__(SEL_THREADS)
pool_hist_kernel(const uint32_t* __restrict__ skey, uint32_t* __restrict__ pkey, uint32_t* __restrict__ ghist0,
                 int64_t max_tokens, int top_k, int eps, SeqMeta meta) {
    __shared__ uint32_t sk[SEL_SLICE + 32];
    __shared__ uint32_t hist[SEL_BINS];
    const int b = blockIdx.y;
    const int tid = threadIdx.x;
    const int l_M = meta.m_end[b] - meta.i_end[b];
    const int base = blockIdx.x * SEL_SLICE;
    if (l_M <= top_k || base >= l_M) return;
    pdl_wait();
    pdl_launch_dependents();
    const uint32_t* src = skey + (int64_t)b * max_tokens;
    for (int i = tid; i < SEL_SLICE + 2 * eps; i += SEL_THREADS) {
        const int m = base - eps + i;
        sk[i] = (m >= 0 && m < l_M) ? __ldcg(src + m) : 0u;
    }
    for (int i = tid; i < SEL_BINS; i += SEL_THREADS) hist[i] = 0u;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < SEL_PER; ++j) {
        const int i = j * SEL_THREADS + tid;
        const int m = base + i;
        uint32_t best = 0u;
        for (int w = 0; w <= 2 * eps; ++w) best = max(best, sk[i + w]);
        const bool valid = m < l_M;
        const uint32_t active = __ballot_sync(0xffffffffu, valid);
        if (valid) {
            pkey[(int64_t)b * max_tokens + m] = best;
            hist_add(hist, best >> 21, active);
        }
    }
    __syncthreads();
    for (int i = tid; i < SEL_BINS; i += SEL_THREADS) {
        const uint32_t c = hist[i];
        if (c) atomicAdd(ghist0 + (int64_t)b * SEL_BINS + i, c);
    }
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

// pooled_ready: ctx->pkey / ctx->ghist0 already hold the pooled keys and their first-digit histogram;
// otherwise ctx->skey holds unpooled keys and ctx->ghist0 is zero.
cudaError_t launch_select(esa_ctx* ctx, int B, bool mapped, const SeqMeta& meta, int max_lM, bool pooled_ready,
                          int32_t* idx_out, int32_t* n_sel_out, cudaStream_t st) {
    const int n_slices = (max_lM + SEL_SLICE - 1) / SEL_SLICE;
    if (n_slices < 1 || n_slices > ctx->sel_slice_stride) return cudaErrorInvalidConfiguration;
    cudaError_t e;
    if (!pooled_ready) {
        ProfScope prof(ctx, KC_POOL_HIST, st);
        e = launch_pdl(pool_hist_kernel, dim3(n_slices, B), dim3(SEL_THREADS), 0, st, (const uint32_t*)ctx->skey, ctx->pkey,
                       ctx->ghist0, ctx->cfg.max_tokens, ctx->cfg.top_k, ctx->cfg.eps, meta);
        if (e != cudaSuccess) return e;
        ctx->launches += 1;
    }
    SelectParams p;
    p.pkey = ctx->pkey; p.ghist0 = ctx->ghist0; p.ghist1 = ctx->ghist1; p.rkey = ctx->rkey;
    p.ckey = ctx->skey; p.cidx = ctx->cidx; p.slice_cnt = ctx->sel_slice_cnt; p.ticket = ctx->sel_ticket;
    p.idx_out = idx_out; p.n_sel_out = n_sel_out;
    p.max_tokens = ctx->cfg.max_tokens; p.slice_stride = ctx->sel_slice_stride; p.top_k = ctx->cfg.top_k;
    p.mapped = mapped ? 1 : 0; p.l_C = 1; p.meta = meta;     // (mapped mode reads rkey[b]: one query per sequence)
    constexpr size_t smem = (size_t)(SEL_MAX_SLICES_SMEM + 2 * SEL_STAGE_CAP) * 4;
    e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    ProfScope prof(ctx, KC_SELECT_TOPK, st);
    e = launch_pdl(select_topk_kernel, dim3(n_slices, B), dim3(SEL_THREADS), smem, st, p);
    if (e != cudaSuccess) return e;
    ctx->launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_select_all(esa_ctx* ctx, int B, const SeqMeta& meta, int32_t* idx_out,
                              int32_t* n_sel_out, cudaStream_t st) {
    int gx = (ctx->cfg.top_k + 255) / 256;
    if (gx > 64) gx = 64;
    if (gx < 1) gx = 1;
    ProfScope prof(ctx, KC_SELECT_ALL, st);
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
