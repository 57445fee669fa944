// Eq. 1 / Algorithm 1: attention of the current chunk over the reduced key set
// I u M_k u L u C, with the K/V gather fused into the tile loads.
//
// The attended keys form a virtual list of n_att = |I| + n_sel + |L| + l_C entries:
//   j in [0, i_end)                      -> token j                       (initial tokens)
//   j in [i_end, i_end + n_sel)          -> token idx[j - i_end]           (selected middle tokens)
//   j >= i_end + n_sel                   -> token m_end + (j - i_end - n_sel)   (L then C, contiguous)
// The last l_C entries are the chunk itself: entry n_att - l_C + u is visible to query c
// iff u <= c (Algorithm 1: causal on [L, C] with bottom-right alignment, everything else
// non-causal).  One softmax spans the whole list, which is what Algorithm 1's two calls
// merged by their log-sum-exp compute when both use the same queries.
//
// Rows of the MMA tile are (query, head-in-group) pairs, row = c * G + g with
// G = H / H_G, so one K/V tile gathered for a key/value head serves all G query heads
// that share it.  Flash-style online softmax in the exp2 domain, bf16 operands, fp32
// scores and accumulators.
//
// This file holds the kernels for small chunks: a generic split-KV mma.sync kernel
// (up to 64 rows per key/value head), the streaming kernel for decode (one query per
// sequence), the kernel that merges the partial (O, m, l) triples of key-list splits -- the
// same algebra as Algorithm 1's merge -- and the entry point that needs no allocation.
// Prefill-sized chunks run in esa_attend_tc.cu.
#include <mutex>

#include "esa_internal.h"

namespace esa {

struct AttendParams {
    const __nv_bfloat16* Q;   // [B, l_C, H, D]
    const __nv_bfloat16* K;   // [B, max_tokens, HG, D]
    const __nv_bfloat16* Qg;  // two-position attention (Section 3.2): queries / keys used against I and M_k
    const __nv_bfloat16* Kg;  //   (equal to Q / K otherwise)
    const __nv_bfloat16* V;
    __nv_bfloat16* O;         // [B, l_C, H, D]
    const int32_t* idx;       // [B, top_k]
    const int32_t* n_sel;     // [B]
    float* part;              // split partials
    int* unit_count;          // arrival counters per (sequence, key/value head) for the in-kernel merge of the decode kernel
    int* status;              // device status word (may be null: the entry point without a context)
    int staged;               // the caches hold the attended list itself: row j = list entry j
    int early;                // the older rows of L may be attended ahead of the wait for the preceding kernel
    int64_t max_tokens;
    int l_C, H, HG, G, top_k;
    int nsplit;
    float scale_log2;         // softmax scale * log2(e)
    SeqMeta meta;
};

// layout of the split-KV partial buffer, per (b, kvh, split): R rows x (D + 2) floats
// (unnormalised O row, running max m in the exp2 domain, running sum l)

// TWO: the list entries of I and M_k (the first n_glob) take their logits from Qg and Kg, the entries
// of L and C from Q and K; both score tiles are formed and each key column keeps the one that applies.
template <int D, int NW, int BN, bool TWO>
__global__ void __launch_bounds__(NW * 32)
attend_kernel(AttendParams p) {
    constexpr int CH = D / 8;
    constexpr int BM = NW * 16;
    constexpr int NT = NW * 32;
    extern __shared__ uint4 smem[];
    uint4* sQ = smem;                         // [BM][CH]
    uint4* sK = sQ + BM * CH;                 // 2 x [BN][CH]
    uint4* sV = sK + 2 * BN * CH;             // 2 x [BN][CH]
    uint4* sQg = sV + 2 * BN * CH;            // [BM][CH] (TWO)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row0 = blockIdx.x * BM;
    const int kvh = blockIdx.y;
    const int b = blockIdx.z / p.nsplit;
    const int split = blockIdx.z % p.nsplit;
    const int G = p.G;
    const int R = p.l_C * G;

    const int t = p.meta.t[b], i_end = p.meta.i_end[b], m_end = p.meta.m_end[b];
    int n_sel = p.n_sel[b];
    n_sel = max(0, min(n_sel, min(p.top_k, m_end - i_end)));
    const int n_glob = i_end + n_sel;                  // entries before L
    const int n_att = n_glob + (t - m_end) + p.l_C;
    const int c_first = n_att - p.l_C;                 // list position of the chunk's first key

    // keys this row tile can see: up to the chunk key of its last query
    const int r_last = min(R, row0 + BM) - 1;
    const int j_end = c_first + r_last / G + 1;
    const int n_tiles = (j_end + BN - 1) / BN;
    const int per = (n_tiles + p.nsplit - 1) / p.nsplit;
    const int tile_begin = split * per;
    const int tile_end = min(n_tiles, tile_begin + per);

    const __nv_bfloat16* Kb = p.K + ((int64_t)b * p.max_tokens * p.HG + kvh) * D;
    const __nv_bfloat16* Kgb = p.Kg + ((int64_t)b * p.max_tokens * p.HG + kvh) * D;
    const __nv_bfloat16* Vb = p.V + ((int64_t)b * p.max_tokens * p.HG + kvh) * D;
    const int32_t* idx = p.idx + (int64_t)b * p.top_k;
    const int64_t tok_stride = (int64_t)p.HG * D;

    int bad_idx = 0;
    auto load_kv = [&](int st, int tile) {
        uint4* dk = sK + st * BN * CH;
        uint4* dv = sV + st * BN * CH;
        for (int i = tid; i < BN * CH; i += NT) {
            int r = i / CH, c = i % CH;
            int j = tile * BN + r;
            bool ok = j < n_att;
            int pos = 0;
            if (ok) {
                if (p.staged) pos = j;
                else if (j < i_end) pos = j;
                else if (j < n_glob) pos = clamp_selected(__ldg(idx + (j - i_end)), i_end, m_end, bad_idx);
                else pos = m_end + (j - n_glob);
            }
            const int64_t off = (int64_t)pos * tok_stride + c * 8;
            cp_async16(&dk[swz<CH>(r, c)], ((TWO && j < n_glob) ? Kgb : Kb) + off, ok ? 16 : 0);
            cp_async16(&dv[swz<CH>(r, c)], Vb + off, ok ? 16 : 0);
        }
    };

    // Q tile -> smem (rows past R are zero)
    for (int i = tid; i < BM * CH; i += NT) {
        int r = i / CH, c = i % CH;
        int row = row0 + r;
        bool ok = row < R;
        int cq = ok ? row / G : 0, g = ok ? row % G : 0;
        const int64_t qoff = (((int64_t)b * p.l_C + cq) * p.H + kvh * G + g) * D + c * 8;
        cp_async16(&sQ[swz<CH>(r, c)], p.Q + qoff, ok ? 16 : 0);
        if (TWO) cp_async16(&sQg[swz<CH>(r, c)], p.Qg + qoff, ok ? 16 : 0);
    }
    if (tile_begin < tile_end) load_kv(0, tile_begin);
    cp_async_commit();

    float o_acc[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) o_acc[i][j] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};

    // this thread's two rows and their causal limits (first invisible list position)
    const int r_lo = row0 + warp * 16 + (lane >> 2);
    const int lim_lo = c_first + min(r_lo / G, p.l_C - 1) + 1;
    const int lim_hi = c_first + min((r_lo + 8) / G, p.l_C - 1) + 1;
    const int warp_min_lim = c_first + min((row0 + warp * 16) / G, p.l_C - 1) + 1;

    uint32_t qf[D / 16][4];
    uint32_t qfg[TWO ? D / 16 : 1][4];
    bool q_loaded = false;

    for (int tile = tile_begin; tile < tile_end; ++tile) {
        const int st = (tile - tile_begin) & 1;
        if (tile + 1 < tile_end) {
            load_kv(st ^ 1, tile + 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (!q_loaded) {
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) load_a_frag<CH>(qf[ks], sQ, warp * 16, ks * 2, lane);
            if (TWO) {
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) load_a_frag<CH>(qfg[ks], sQg, warp * 16, ks * 2, lane);
            }
            q_loaded = true;
        }
        const uint4* tk = sK + st * BN * CH;
        const uint4* tv = sV + st * BN * CH;

        // S = Q K^T
        float s[BN / 8][4];
#pragma unroll
        for (int i = 0; i < BN / 8; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
            for (int nb = 0; nb < BN / 16; ++nb) {
                uint32_t kb[4];
                load_b_frag_nk<CH>(kb, tk, nb * 16, ks * 2, lane);
                mma_bf16_16816(s[2 * nb], qf[ks], kb[0], kb[1]);
                mma_bf16_16816(s[2 * nb + 1], qf[ks], kb[2], kb[3]);
            }
        }
        const int j0 = tile * BN;
        if (TWO && j0 < n_glob) {
            // some key columns of this tile belong to I or M_k: their logits come from Qg (the tile holds Kg rows there)
            float sg[BN / 8][4];
#pragma unroll
            for (int i = 0; i < BN / 8; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) sg[i][j] = 0.f;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
                for (int nb = 0; nb < BN / 16; ++nb) {
                    uint32_t kb[4];
                    load_b_frag_nk<CH>(kb, tk, nb * 16, ks * 2, lane);
                    mma_bf16_16816(sg[2 * nb], qfg[ks], kb[0], kb[1]);
                    mma_bf16_16816(sg[2 * nb + 1], qfg[ks], kb[2], kb[3]);
                }
            }
#pragma unroll
            for (int nb = 0; nb < BN / 8; ++nb)
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    if (j0 + nb * 8 + (lane & 3) * 2 + e < n_glob) {
                        s[nb][e] = sg[nb][e];
                        s[nb][2 + e] = sg[nb][2 + e];
                    }
        }

        // scale, mask (causal inside C and the ragged tail), online softmax
        const bool need_mask = j0 + BN > warp_min_lim;
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int nb = 0; nb < BN / 8; ++nb) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float a = s[nb][e] * p.scale_log2, c2 = s[nb][2 + e] * p.scale_log2;
                if (need_mask) {
                    int j = j0 + nb * 8 + (lane & 3) * 2 + e;
                    if (j >= lim_lo) a = -INFINITY;
                    if (j >= lim_hi) c2 = -INFINITY;
                }
                s[nb][e] = a;
                s[nb][2 + e] = c2;
                mx_lo = fmaxf(mx_lo, a);
                mx_hi = fmaxf(mx_hi, c2);
            }
        }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
        const float mn_lo = fmaxf(m_run[0], mx_lo), mn_hi = fmaxf(m_run[1], mx_hi);
        const float ms_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo;   // a fully masked row stays empty
        const float ms_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
        const float al_lo = fast_exp2(m_run[0] - ms_lo), al_hi = fast_exp2(m_run[1] - ms_hi);
        m_run[0] = mn_lo;
        m_run[1] = mn_hi;
        float sum_lo = 0.f, sum_hi = 0.f;
        uint32_t pf[BN / 16][4];
#pragma unroll
        for (int nb = 0; nb < BN / 8; ++nb) {
            float p0 = fast_exp2(s[nb][0] - ms_lo), p1 = fast_exp2(s[nb][1] - ms_lo);
            float p2 = fast_exp2(s[nb][2] - ms_hi), p3 = fast_exp2(s[nb][3] - ms_hi);
            sum_lo += p0 + p1;
            sum_hi += p2 + p3;
            pf[nb >> 1][(nb & 1) * 2] = pack_bf16(p0, p1);
            pf[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
        l_run[0] = l_run[0] * al_lo + sum_lo;
        l_run[1] = l_run[1] * al_hi + sum_hi;
#pragma unroll
        for (int nb = 0; nb < D / 8; ++nb) {
            o_acc[nb][0] *= al_lo;
            o_acc[nb][1] *= al_lo;
            o_acc[nb][2] *= al_hi;
            o_acc[nb][3] *= al_hi;
        }
        // O += P V
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk) {
#pragma unroll
            for (int dp = 0; dp < D / 16; ++dp) {
                uint32_t vb[4];
                load_b_frag_kn<CH>(vb, tv, kk * 16, dp * 2, lane);
                mma_bf16_16816(o_acc[2 * dp], pf[kk], vb[0], vb[1]);
                mma_bf16_16816(o_acc[2 * dp + 1], pf[kk], vb[2], vb[3]);
            }
        }
        __syncthreads();
    }
    cp_async_wait<0>();
    if (bad_idx && p.status) atomicExch(p.status, kStatusBadIndex);

    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);

#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int row = r_lo + half * 8;
        if (row >= R) continue;
        if (p.nsplit == 1) {
            const float inv = 1.f / l_run[half];
            const int cq = row / G, g = row % G;
            __nv_bfloat16* dst = p.O + (((int64_t)b * p.l_C + cq) * p.H + kvh * G + g) * D;
#pragma unroll
            for (int nb = 0; nb < D / 8; ++nb) {
                int col = nb * 8 + (lane & 3) * 2;
                *reinterpret_cast<uint32_t*>(dst + col) =
                    pack_bf16(o_acc[nb][half * 2] * inv, o_acc[nb][half * 2 + 1] * inv);
            }
        } else {
            float* dst = p.part + ((((int64_t)b * p.HG + kvh) * p.nsplit + split) * R + row) * (D + 2);
#pragma unroll
            for (int nb = 0; nb < D / 8; ++nb) {
                int col = nb * 8 + (lane & 3) * 2;
                *reinterpret_cast<float2*>(dst + col) = make_float2(o_acc[nb][half * 2], o_acc[nb][half * 2 + 1]);
            }
            if ((lane & 3) == 0) {
                dst[D] = m_run[half];
                dst[D + 1] = l_run[half];
            }
        }
    }
}

// Merge of the split-KV partials (Algorithm 1's merge generalised to nsplit parts):
// O = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s with M = max_s m_s.
// One warp per output row: each lane owns D / 32 consecutive columns, so a part's row is one
// coalesced read and the result one coalesced bf16 write.
// Combines the nsplit parts of one row (Algorithm 1's merge of (O, m, l)) and writes the bf16 row.
// `base` points at the row's slot in part 0, parts are `sstride` floats apart.  Loads go to L2
// (the parts may have been written by other SMs a moment ago).
template <int D>
__device__ __forceinline__ void merge_row(const float* base, int64_t sstride, int nsplit, int lane, __nv_bfloat16* dst_row) {
    constexpr int PER = D / 32;                  // columns per lane: 2 or 4
    // parts are taken four at a time so that their loads are in flight together
    float M = -INFINITY;
    for (int s = 0; s < nsplit; ++s) M = fmaxf(M, __ldcg(base + s * sstride + D));
    float den = 0.f;
    float acc[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) acc[i] = 0.f;
    for (int s0 = 0; s0 < nsplit; s0 += 4) {
        float mm[4], ll[4];
        float2 v[4][PER / 2];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bool in = s0 + j < nsplit;
            const float* ps = base + (in ? s0 + j : 0) * sstride;
            mm[j] = in ? __ldcg(ps + D) : -INFINITY;
            ll[j] = __ldcg(ps + D + 1);
#pragma unroll
            for (int i = 0; i < PER / 2; ++i) v[j][i] = __ldcg(reinterpret_cast<const float2*>(ps + lane * PER + 2 * i));
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (mm[j] == -INFINITY) continue;        // an empty or absent part (uniform over the warp)
            const float w = fast_exp2(mm[j] - M);
            den += w * ll[j];
#pragma unroll
            for (int i = 0; i < PER / 2; ++i) {
                acc[2 * i] += w * v[j][i].x;
                acc[2 * i + 1] += w * v[j][i].y;
            }
        }
    }
    const float inv = 1.f / den;
#pragma unroll
    for (int i = 0; i < PER; i += 2)
        *reinterpret_cast<uint32_t*>(dst_row + lane * PER + i) = pack_bf16(acc[i] * inv, acc[i + 1] * inv);
}

template <int D>
__global__ void __launch_bounds__(256) attend_merge_kernel(AttendParams p) {
    pdl_wait();
    pdl_launch_dependents();
    const int R = p.l_C * p.G;
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int kvh = blockIdx.y, b = blockIdx.z;
    if (row >= R) return;
    const float* base = p.part + (((int64_t)b * p.HG + kvh) * p.nsplit * R + row) * (D + 2);
    const int cq = row / p.G, g = row % p.G;
    merge_row<D>(base, (int64_t)R * (D + 2), p.nsplit, lane, p.O + (((int64_t)b * p.l_C + cq) * p.H + kvh * p.G + g) * D);
}

// ---------------------------------------------------------------------------
// Decode (one query per sequence): the step is bound by reading the gathered K/V rows, so the
// kernel is built around the stream of rows, not around the arithmetic.  Every warp pulls its
// rows through a private ring of shared-memory stages filled by index-driven 16-byte cp.async
// (16 rows of K and of V per stage, DEC_STAGES - 1 stages in flight per warp, the positions
// looked up one iteration further ahead).  The arithmetic runs on mma.sync with the rows on the
// 16-wide M side -- S^T = K Q^T and O^T += V^T P^T -- so that the G <= 8 heads of the group sit
// on the 8-wide N side: no padding along the long dimension and ~65 instructions per 16 rows.
// Warps and key-list splits are merged with the (O, m, l) algebra of Algorithm 1's merge.
// ---------------------------------------------------------------------------
constexpr int DEC_WARPS = 4;
constexpr int DEC_STAGES = 3;
constexpr int DEC_ROWS = 16;       // rows (keys) per stage

template <int D, int G, bool TWO>
__global__ void __launch_bounds__(DEC_WARPS * 32)
attend_decode_kernel(AttendParams p) {
    constexpr int CH = D / 8;                        // 16-byte chunks per row
    constexpr int TILE_CHUNKS = DEC_ROWS * CH;       // one K or V tile, in chunks
    constexpr int STAGE_CHUNKS = 2 * TILE_CHUNKS;
    constexpr int PER_LANE = TILE_CHUNKS / 32;       // chunk copies per lane and tile
    constexpr int ROWS_PER_PASS = 32 / CH;           // rows covered by one copy instruction of the warp
    static_assert(G <= 8, "the heads of a group sit on the 8-wide side of the MMA");
    extern __shared__ uint4 dec_smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    uint4* ring = dec_smem + warp * (DEC_STAGES * STAGE_CHUNKS);

    // The rows of L that are older than this step's token do not depend on the selection, nor on anything the
    // preceding kernels of the step wrote: every CTA attends its share of them BEFORE the wait for the preceding
    // kernel (phase 0, positions counted within L u C: cache row m_end + u), while the selection kernel is
    // still at work on a handful of SMs, and its share of the rest of the list after it (phase 1, list positions).
    // (Not with two position encodings, nor when the caches hold the staged list: phase 1 alone does everything.)
    const int t = p.meta.t[b], i_end = p.meta.i_end[b], m_end = p.meta.m_end[b];
    const bool early = !TWO && p.early;
    const int u_pre = early ? ((t - m_end) / DEC_ROWS) * DEC_ROWS : 0;     // rows of L done in phase 0: whole iterations
    const int itA_all = u_pre / DEC_ROWS;
    const int perA = (itA_all + p.nsplit - 1) / p.nsplit;
    const int itA_begin = min(itA_all, split * perA), itA_end = min(itA_all, itA_begin + perA);
    // phase 1, set after the wait
    int n_glob = 0, n_att = 0, itF = 0, itT = 0;

    const int my_chunk = lane % CH, my_row = lane / CH;     // copies of this lane: rows my_row + i * ROWS_PER_PASS
    const __nv_bfloat16* Kb = p.K + ((int64_t)b * p.max_tokens * p.HG + kvh) * D + my_chunk * 8;
    const __nv_bfloat16* Kgb = p.Kg + ((int64_t)b * p.max_tokens * p.HG + kvh) * D + my_chunk * 8;
    const __nv_bfloat16* Vb = p.V + ((int64_t)b * p.max_tokens * p.HG + kvh) * D + my_chunk * 8;
    const int32_t* idx = p.idx + (int64_t)b * p.top_k;
    const int64_t tok_stride = (int64_t)p.HG * D;

    // Phase 1 walks the iterations (16 list positions each) that still hold a row to attend: those below
    // itF = ceil(n_glob / 16) (I and M_k) and those from itT on (the rows of L u C left for this phase).
    auto iter_of = [&](int ph, int v) { return (ph == 0 || v < itF) ? v : itT + (v - itF); };
    auto row_valid = [&](int ph, int j) { return ph == 0 || (j < n_att && !(j >= n_glob && j < n_glob + u_pre)); };

    // list positions -> token positions of the rows of iteration `v` that this lane copies
    // (a position read from the selection is range-checked when it is used, one iteration later, so that
    // the index load stays in flight meanwhile; sel_mask remembers which rows those are)
    int bad_idx = 0;
    uint32_t sel_mask = 0;          // rows of the positions looked up last that came from the selection
    uint32_t far_mask = 0;          // rows of the positions looked up last that belong to I or M_k (TWO: their keys come from Kg)
    auto lookup = [&](int ph, int v, int v_end, int (&pos)[PER_LANE]) {
        sel_mask = 0;
        far_mask = 0;
        const int it = iter_of(ph, v);
#pragma unroll
        for (int i = 0; i < PER_LANE; ++i) {
            const int j = it * DEC_ROWS + my_row + i * ROWS_PER_PASS;
            int q = -1;
            if (v < v_end) {
                if (ph == 0) q = m_end + j;
                else if (row_valid(1, j)) {
                    if (TWO && j < n_glob) far_mask |= 1u << i;
                    if (p.staged || j < i_end) q = j;
                    else if (j < n_glob) {
                        q = __ldg(idx + (j - i_end));
                        sel_mask |= 1u << i;
                    } else q = m_end + (j - n_glob);
                }
            }
            pos[i] = q;
        }
    };
    auto issue = [&](int stage, int (&pos)[PER_LANE], uint32_t mask, uint32_t fmask) {
        uint4* sk = ring + stage * STAGE_CHUNKS;
        uint4* sv = sk + TILE_CHUNKS;
#pragma unroll
        for (int i = 0; i < PER_LANE; ++i) {
            const int r = my_row + i * ROWS_PER_PASS;
            int q = pos[i];
            if ((mask >> i) & 1u) q = clamp_selected(q, i_end, m_end, bad_idx);
            const int64_t off = (int64_t)(q < 0 ? 0 : q) * tok_stride;
            cp_async16(&sk[swz<CH>(r, my_chunk)], ((TWO && ((fmask >> i) & 1u)) ? Kgb : Kb) + off, q < 0 ? 0 : 16);
            cp_async16(&sv[swz<CH>(r, my_chunk)], Vb + off, q < 0 ? 0 : 16);
        }
    };

    // B fragments of Q^T for every 16-wide slice of D: element (k = d, n = head); heads >= G are zero
    uint32_t qb[D / 16][2];
    uint32_t qbg[TWO ? D / 16 : 1][2];      // the same for the queries used against I and M_k
    {
        const int head = lane >> 2;
        const int64_t qoff = ((int64_t)b * p.H + kvh * G + (head < G ? head : 0)) * D;
        const __nv_bfloat16* qrow = p.Q + qoff;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            const int d0 = ks * 16 + 2 * (lane & 3);
            qb[ks][0] = head < G ? *reinterpret_cast<const uint32_t*>(qrow + d0) : 0u;
            qb[ks][1] = head < G ? *reinterpret_cast<const uint32_t*>(qrow + d0 + 8) : 0u;
            if (TWO) {
                qbg[ks][0] = head < G ? *reinterpret_cast<const uint32_t*>(p.Qg + qoff + d0) : 0u;
                qbg[ks][1] = head < G ? *reinterpret_cast<const uint32_t*>(p.Qg + qoff + d0 + 8) : 0u;
            }
        }
    }
    // this thread's two heads (columns 2 (lane & 3), +1): running maximum and its share of the sum;
    // O^T: D / 16 tiles of (16 values of d) x (8 heads), c-fragment layout
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o_acc[D / 16][4];
#pragma unroll
    for (int i = 0; i < D / 16; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) o_acc[i][j] = 0.f;

#pragma unroll 1
    for (int ph = 0; ph < 2; ++ph) {
        int v_begin, v_end;
        if (ph == 0) {
            v_begin = itA_begin;
            v_end = itA_end;
        } else {
            // everything the selection wrote (n_sel, idx), and rows that may have been appended by the kernel before
            pdl_wait();
            pdl_launch_dependents();
            int n_sel = p.n_sel[b];
            n_sel = max(0, min(n_sel, min(p.top_k, m_end - i_end)));
            n_glob = i_end + n_sel;
            n_att = n_glob + (t - m_end) + 1;            // the single query sees every listed key
            const int iters_all = (n_att + DEC_ROWS - 1) / DEC_ROWS;
            itF = (n_glob + DEC_ROWS - 1) / DEC_ROWS;
            itT = max(itF, (n_glob + u_pre) / DEC_ROWS);
            const int v_all = itF + max(0, iters_all - itT);
            const int per = (v_all + p.nsplit - 1) / p.nsplit;
            v_begin = min(v_all, split * per);
            v_end = min(v_all, v_begin + per);
        }
        // prologue: DEC_STAGES - 1 iterations in flight, positions of one more in registers
        int pos_next[PER_LANE];
        const int v0 = v_begin + warp;
#pragma unroll
        for (int s = 0; s < DEC_STAGES - 1; ++s) {
            lookup(ph, v0 + s * DEC_WARPS, v_end, pos_next);
            issue(s, pos_next, sel_mask, far_mask);
            cp_async_commit();
        }
        lookup(ph, v0 + (DEC_STAGES - 1) * DEC_WARPS, v_end, pos_next);

        int n = 0;
        for (int v = v0; v < v_end; v += DEC_WARPS, ++n) {
            issue((n + DEC_STAGES - 1) % DEC_STAGES, pos_next, sel_mask, far_mask);
            cp_async_commit();
            lookup(ph, v + DEC_STAGES * DEC_WARPS, v_end, pos_next);
            cp_async_wait<DEC_STAGES - 1>();
            __syncwarp();
            const uint4* tk = ring + (n % DEC_STAGES) * STAGE_CHUNKS;
            const uint4* tv = tk + TILE_CHUNKS;

            // S^T[key, head] = K Q^T
            float sc[4] = {0.f, 0.f, 0.f, 0.f};
    #pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                uint32_t a[4];
                load_a_frag<CH>(a, tk, 0, ks * 2, lane);
                mma_bf16_16816(sc, a, qb[ks][0], qb[ks][1]);
            }
            // rows lane / 4 and + 8 of the tile; list positions past the end are masked
            const int it = iter_of(ph, v);
            const int key_lo = it * DEC_ROWS + (lane >> 2);
            if (TWO && it * DEC_ROWS < n_glob) {
                // rows of I and M_k: logits against the other query encoding (uniform branch over the warp)
                float sg[4] = {0.f, 0.f, 0.f, 0.f};
    #pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    uint32_t a[4];
                    load_a_frag<CH>(a, tk, 0, ks * 2, lane);
                    mma_bf16_16816(sg, a, qbg[ks][0], qbg[ks][1]);
                }
                if (key_lo < n_glob) { sc[0] = sg[0]; sc[1] = sg[1]; }
                if (key_lo + 8 < n_glob) { sc[2] = sg[2]; sc[3] = sg[3]; }
            }
            const bool ok_lo = row_valid(ph, key_lo), ok_hi = row_valid(ph, key_lo + 8);
            sc[0] = ok_lo ? sc[0] * p.scale_log2 : -INFINITY;
            sc[1] = ok_lo ? sc[1] * p.scale_log2 : -INFINITY;
            sc[2] = ok_hi ? sc[2] * p.scale_log2 : -INFINITY;
            sc[3] = ok_hi ? sc[3] * p.scale_log2 : -INFINITY;
            float mx0 = fmaxf(sc[0], sc[2]), mx1 = fmaxf(sc[1], sc[3]);
    #pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
            }
            const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
            const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
            if (mn0 != m_run[0] || mn1 != m_run[1]) {          // uniform over the lanes that share the heads
                const float al0 = fast_exp2(m_run[0] - ms0), al1 = fast_exp2(m_run[1] - ms1);
                l_run[0] *= al0;
                l_run[1] *= al1;
    #pragma unroll
                for (int i = 0; i < D / 16; ++i) {
                    o_acc[i][0] *= al0; o_acc[i][1] *= al1; o_acc[i][2] *= al0; o_acc[i][3] *= al1;
                }
                m_run[0] = mn0;
                m_run[1] = mn1;
            }
            const float p0 = fast_exp2(sc[0] - ms0), p1 = fast_exp2(sc[1] - ms1);
            const float p2 = fast_exp2(sc[2] - ms0), p3 = fast_exp2(sc[3] - ms1);
            l_run[0] += p0 + p2;
            l_run[1] += p1 + p3;
            // P^T as the B operand (k = key, n = head): thread T needs keys 2 (T & 3), +1 (and + 8) of head T / 4;
            // in the accumulator layout those sit in lanes (key & 7) * 4 + head / 2, packed per head pair.
            const uint32_t w_lo = pack_bf16(p0, p1), w_hi = pack_bf16(p2, p3);       // keys r and r + 8, heads 2q, 2q + 1
            const int src0 = (2 * (lane & 3)) * 4 + (lane >> 3), src1 = src0 + 4;
            const uint32_t a_lo = __shfl_sync(0xffffffffu, w_lo, src0), b_lo = __shfl_sync(0xffffffffu, w_lo, src1);
            const uint32_t a_hi = __shfl_sync(0xffffffffu, w_hi, src0), b_hi = __shfl_sync(0xffffffffu, w_hi, src1);
            const uint32_t sel = ((lane >> 2) & 1) ? 0x7632u : 0x5410u;               // odd head: upper halves, else lower
            const uint32_t pb0 = __byte_perm(a_lo, b_lo, sel), pb1 = __byte_perm(a_hi, b_hi, sel);
            // O^T[d, head] += V^T P^T: A = V^T from the row-major V tile through transposing ldmatrix
    #pragma unroll
            for (int dt = 0; dt < D / 16; ++dt) {
                uint32_t av[4];
                const int r = (lane & 7) + ((lane >> 4) & 1) * 8;          // key row of this lane's matrix
                const int c = dt * 2 + ((lane >> 3) & 1);                 // 16-byte chunk: d 0-7 or 8-15 of the tile
                ldmatrix_x4_trans(av, tv + swz<CH>(r, c));
                mma_bf16_16816(o_acc[dt], av, pb0, pb1);
            }
            __syncwarp();          // the stage is free for the copy issued next iteration
        }
        cp_async_wait<0>();
        __syncwarp();
    }
    cp_async_wait<0>();
    if (bad_idx && p.status) atomicExch(p.status, kStatusBadIndex);

    // the lanes that share a head pair (same lane & 3) each saw different rows: add their sums
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], o);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], o);
    }
    // merge the warps through shared memory (the rings are idle now)
    __syncthreads();
    float* s_m = reinterpret_cast<float*>(dec_smem);          // [DEC_WARPS][8]
    float* s_l = s_m + DEC_WARPS * 8;                          // [DEC_WARPS][8]
    float* s_acc = s_l + DEC_WARPS * 8;                        // [DEC_WARPS][8][D]
    {
        const int h0 = 2 * (lane & 3);
        if (lane < 4) {
            s_m[warp * 8 + h0] = m_run[0]; s_m[warp * 8 + h0 + 1] = m_run[1];
            s_l[warp * 8 + h0] = l_run[0]; s_l[warp * 8 + h0 + 1] = l_run[1];
        }
#pragma unroll
        for (int dt = 0; dt < D / 16; ++dt) {
            const int d0 = dt * 16 + (lane >> 2);
            s_acc[(warp * 8 + h0) * D + d0] = o_acc[dt][0];
            s_acc[(warp * 8 + h0 + 1) * D + d0] = o_acc[dt][1];
            s_acc[(warp * 8 + h0) * D + d0 + 8] = o_acc[dt][2];
            s_acc[(warp * 8 + h0 + 1) * D + d0 + 8] = o_acc[dt][3];
        }
    }
    __syncthreads();
    // thread (g, column) combines the DEC_WARPS parts
    for (int e = tid; e < G * D; e += DEC_WARPS * 32) {
        const int g = e / D, col = e % D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, s_m[w * 8 + g]);
        const float Ms = (M == -INFINITY) ? 0.f : M;
        float o = 0.f, lsum = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) {
            const float wgt = fast_exp2(s_m[w * 8 + g] - Ms);
            o += wgt * s_acc[(w * 8 + g) * D + col];
            lsum += wgt * s_l[w * 8 + g];
        }
        if (p.nsplit == 1) {
            p.O[((int64_t)b * p.H + kvh * G + g) * D + col] = __float2bfloat16_rn(o / lsum);
        } else {
            float* dst = p.part + ((((int64_t)b * p.HG + kvh) * p.nsplit + split) * G + g) * (D + 2);
            dst[col] = o;
            if (col == 0) { dst[D] = M; dst[D + 1] = lsum; }
        }
    }
    if (p.nsplit > 1) {
        // The CTA that completes a (sequence, key/value head) unit merges its parts: an arrival
        // counter decides, nobody waits, and the counter returns to 0 for the next launch.
        __shared__ int s_last;
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            int* cnt = p.unit_count + b * p.HG + kvh;
            const int ticket = atomicAdd(cnt, 1);
            s_last = ticket == p.nsplit - 1;
            if (s_last) *cnt = 0;
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            for (int g = warp; g < G; g += DEC_WARPS) {
                const float* base = p.part + (((int64_t)b * p.HG + kvh) * p.nsplit * G + g) * (D + 2);
                merge_row<D>(base, (int64_t)G * (D + 2), p.nsplit, lane, p.O + ((int64_t)b * p.H + kvh * G + g) * D);
            }
        }
    }
}

template <int D, int G, bool TWO>
static cudaError_t launch_decode_t(esa_ctx* ctx, AttendParams& p, int B, int n_att_max, cudaStream_t st) {
    constexpr int smem = DEC_WARPS * DEC_STAGES * 2 * DEC_ROWS * D * 2;
    static_assert(smem >= (2 * DEC_WARPS * 8 + DEC_WARPS * 8 * D) * 4, "the warp merge reuses the rings");
    cudaError_t e = cudaFuncSetAttribute(attend_decode_kernel<D, G, TWO>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int per_sm = 1;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attend_decode_kernel<D, G, TWO>, DEC_WARPS * 32, smem);
    if (e != cudaSuccess) return e;
    const int iters = (n_att_max + DEC_ROWS - 1) / DEC_ROWS;
    // one wave of CTAs, each warp with at least a few iterations
    int nsplit = (per_sm * ctx->num_sms) / (p.HG * B);
    if (nsplit > kAttMaxSplits) nsplit = kAttMaxSplits;
    if (nsplit > (iters + 4 * DEC_WARPS - 1) / (4 * DEC_WARPS)) nsplit = (iters + 4 * DEC_WARPS - 1) / (4 * DEC_WARPS);
    while (nsplit > 1 && (size_t)B * p.HG * nsplit * G * (D + 2) > ctx->att_part_elems) --nsplit;
    if (nsplit < 1) nsplit = 1;
    p.nsplit = nsplit;
    if ((size_t)B * p.HG > ctx->att_count_elems) return cudaErrorInvalidConfiguration;
    p.unit_count = ctx->att_count;
    ProfScope prof(ctx, KC_ATTEND_DECODE, st);
    e = launch_pdl(attend_decode_kernel<D, G, TWO>, dim3(nsplit, p.HG, B), dim3(DEC_WARPS * 32), smem, st, p);
    ctx->launches += 1;
    return e;
}

template <int D, bool TWO>
static cudaError_t launch_decode(esa_ctx* ctx, AttendParams& p, int B, int n_att_max, cudaStream_t st) {
    switch (p.G) {
        case 1: return launch_decode_t<D, 1, TWO>(ctx, p, B, n_att_max, st);
        case 2: return launch_decode_t<D, 2, TWO>(ctx, p, B, n_att_max, st);
        case 4: return launch_decode_t<D, 4, TWO>(ctx, p, B, n_att_max, st);
        case 7: return launch_decode_t<D, 7, TWO>(ctx, p, B, n_att_max, st);
        case 8: return launch_decode_t<D, 8, TWO>(ctx, p, B, n_att_max, st);
    }
    return cudaErrorNotSupported;
}

template <int D, int NW, int BN, bool TWO>
static cudaError_t launch_attend_t(esa_ctx* ctx, AttendParams& p, int B, int n_att_max, cudaStream_t st) {
    constexpr int BM = NW * 16;
    const int R = p.l_C * p.G;
    const int row_tiles = (R + BM - 1) / BM;
    constexpr int smem = ((TWO ? 2 : 1) * BM + 4 * BN) * (D / 8) * 16;
    cudaError_t e = cudaFuncSetAttribute(attend_kernel<D, NW, BN, TWO>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int nsplit = 1;
    if (R <= kAttSplitRows && row_tiles == 1) {
        // split the key list so that one wave of CTAs fills the machine (never a second, short wave)
        int per_sm = 1;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attend_kernel<D, NW, BN, TWO>, NW * 32, smem);
        if (e != cudaSuccess) return e;
        const int ctas = p.HG * B;
        const int n_tiles = (n_att_max + BN - 1) / BN;
        nsplit = (per_sm * ctx->num_sms) / ctas;
        if (nsplit > kAttMaxSplits) nsplit = kAttMaxSplits;
        if (nsplit > n_tiles) nsplit = n_tiles;
        while (nsplit > 1 && (size_t)B * p.HG * nsplit * R * (D + 2) > ctx->att_part_elems) --nsplit;
        if (nsplit < 1) nsplit = 1;
    }
    p.nsplit = nsplit;
    {
        ProfScope prof(ctx, KC_ATTEND_SMALL, st);
        attend_kernel<D, NW, BN, TWO><<<dim3(row_tiles, p.HG, B * nsplit), NW * 32, smem, st>>>(p);
    }
    ctx->launches += 1;
    if (nsplit > 1) {
        ProfScope prof(ctx, KC_ATTEND_MERGE, st);
        attend_merge_kernel<D><<<dim3((R + 7) / 8, p.HG, B), 256, 0, st>>>(p);
        ctx->launches += 1;
    }
    return cudaGetLastError();
}

template <bool TWO>
static cudaError_t launch_small(esa_ctx* ctx, AttendParams& p, int B, int l_C, int n_att_max, cudaStream_t st) {
    const int R = l_C * ctx->G;
    if (l_C == 1) {
        // decode: streaming kernel for the usual group sizes
        cudaError_t e = ctx->d == 128 ? launch_decode<128, TWO>(ctx, p, B, n_att_max, st)
                                      : launch_decode<64, TWO>(ctx, p, B, n_att_max, st);
        if (e != cudaErrorNotSupported) return e;
    }
    if (ctx->d == 128) {
        if (R <= 16) return launch_attend_t<128, 1, 32, TWO>(ctx, p, B, n_att_max, st);
        if (R <= 64) return launch_attend_t<128, 4, 64, TWO>(ctx, p, B, n_att_max, st);
        return launch_attend_t<128, 8, 64, TWO>(ctx, p, B, n_att_max, st);
    } else if (ctx->d == 64) {
        if (R <= 16) return launch_attend_t<64, 1, 32, TWO>(ctx, p, B, n_att_max, st);
        if (R <= 64) return launch_attend_t<64, 4, 64, TWO>(ctx, p, B, n_att_max, st);
        return launch_attend_t<64, 8, 64, TWO>(ctx, p, B, n_att_max, st);
    }
    return cudaErrorInvalidValue;
}

// Qg / Kg: queries and key cache used against I and M_k (Section 3.2); null = Q / K.
cudaError_t launch_attend(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* Q, const __nv_bfloat16* Qg,
                          const __nv_bfloat16* K, const __nv_bfloat16* Kg, const __nv_bfloat16* V, const SeqMeta& meta,
                          const int32_t* idx, const int32_t* n_sel, __nv_bfloat16* O, cudaStream_t st, int64_t cache_rows,
                          bool staged) {
    const bool two = (Qg && Qg != Q) || (Kg && Kg != K);
    AttendParams p;
    p.Q = Q; p.K = K; p.Qg = Qg ? Qg : Q; p.Kg = Kg ? Kg : K;
    p.V = V; p.O = O; p.idx = idx; p.n_sel = n_sel; p.part = ctx->att_part; p.unit_count = nullptr;
    p.status = ctx->status;
    p.staged = staged ? 1 : 0;
    p.early = ctx->attend_early && !two && !staged ? 1 : 0;
    p.max_tokens = cache_rows > 0 ? cache_rows : ctx->cfg.max_tokens; p.l_C = l_C; p.H = ctx->H; p.HG = ctx->HG; p.G = ctx->G;
    p.top_k = ctx->cfg.top_k; p.nsplit = 1;
    p.scale_log2 = ctx->scale * 1.4426950408889634f;
    p.meta = meta;
    int n_att_max = 0;
    for (int b = 0; b < B; ++b) {
        int lM = meta.m_end[b] - meta.i_end[b];
        int n = meta.i_end[b] + (lM < ctx->cfg.top_k ? lM : ctx->cfg.top_k) + (meta.t[b] - meta.m_end[b]) + l_C;
        if (n > n_att_max) n_att_max = n;
    }
    const int R = l_C * ctx->G;
    if (R > kAttSplitRows) {
        // prefill-sized chunks: tcgen05 kernel (a split key list is merged inside it)
        int nsplit = 1;
        return launch_attend_tc(ctx, B, l_C, Q, two ? p.Qg : nullptr, K, two ? p.Kg : nullptr, V, meta, idx, n_sel, O, n_att_max, st,
                                &nsplit, cache_rows, staged);
    }
    return two ? launch_small<true>(ctx, p, B, l_C, n_att_max, st) : launch_small<false>(ctx, p, B, l_C, n_att_max, st);
}

// ---------------------------------------------------------------------------
// esa_attend_noalloc: split-key attention of small chunks whose scratch is a fixed array
// that is part of the library image, for callers that must not allocate device memory.
// ---------------------------------------------------------------------------
namespace {

// Partial (O, m, l) rows of the key-list splits.  8 MiB, resident on every GPU that loads
// the library, until the process exits.  Every slot the merge reads is written earlier in
// the same call, so nothing has to be cleared between calls.
constexpr size_t kNoAllocPartFloats = size_t(2) << 20;
static __device__ __align__(256) float g_noalloc_part[kNoAllocPartFloats];

constexpr int kNoAllocMaxDevices = 64;
constexpr int kNoAllocMinSplits = 4;      // a call must be able to split its key list at least this far

struct NoAllocDevice {
    float* part;      // device address of g_noalloc_part on this device (the symbol itself is not one)
    int num_sms;
    bool ready;
};
NoAllocDevice g_noalloc_dev[kNoAllocMaxDevices];
std::mutex g_noalloc_mutex;      // host threads may make a device's first call together

template <int D, int NW, int BN>
cudaError_t launch_noalloc_t(const NoAllocDevice& dev, AttendParams& p, int B, int n_att_max, cudaStream_t st) {
    const int R = p.l_C * p.G;
    constexpr int smem = (NW * 16 + 4 * BN) * (D / 8) * 16;
    cudaError_t e = cudaFuncSetAttribute(attend_kernel<D, NW, BN, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int per_sm = 1;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attend_kernel<D, NW, BN, false>, NW * 32, smem);
    if (e != cudaSuccess) return e;
    const int n_tiles = (n_att_max + BN - 1) / BN;
    int nsplit = (per_sm * dev.num_sms) / (p.HG * B);
    if (nsplit > kAttMaxSplits) nsplit = kAttMaxSplits;
    if (nsplit > n_tiles) nsplit = n_tiles;
    while (nsplit > 1 && (size_t)B * p.HG * nsplit * R * (D + 2) > kNoAllocPartFloats) --nsplit;
    if (nsplit < 1) nsplit = 1;
    p.nsplit = nsplit;
    attend_kernel<D, NW, BN, false><<<dim3(1, p.HG, B * nsplit), NW * 32, smem, st>>>(p);
    if (nsplit > 1) attend_merge_kernel<D><<<dim3((R + 7) / 8, p.HG, B), 256, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace
}  // namespace esa

extern "C" esa_status esa_attend_noalloc(const esa_config* cfg, int32_t B, const void* Q_cur, int32_t l_C,
                                         const void* K_cache, const void* V_cache, const int64_t* n_prev,
                                         const int32_t* idx, const int32_t* n_sel, void* O, void* stream) {
    using namespace esa;
    if (!cfg || !Q_cur || !K_cache || !V_cache || !n_prev || !idx || !n_sel || !O || B <= 0 || l_C <= 0)
        return ESA_ERR_INVALID_ARG;
    if (cfg->n_q_heads <= 0 || cfg->n_kv_heads <= 0 || cfg->n_q_heads % cfg->n_kv_heads ||
        (cfg->head_dim != 64 && cfg->head_dim != 128) || cfg->l_init < 0 || cfg->l_local < 0 || cfg->top_k <= 0 ||
        cfg->max_tokens <= 0 || cfg->max_tokens >= (int64_t(1) << 31) || !(cfg->softmax_scale >= 0.f))
        return ESA_ERR_SHAPE;
    if (B > kMaxBatch) return ESA_ERR_CAPACITY;
    const int G = cfg->n_q_heads / cfg->n_kv_heads, D = cfg->head_dim;
    const int64_t R = (int64_t)l_C * G;
    // only the split-key kernel of small chunks has a scratch-backed variant here
    if (R > kAttSplitRows) return ESA_ERR_CAPACITY;
    // the fixed array must leave room for at least kNoAllocMinSplits parts
    if ((size_t)B * cfg->n_kv_heads * kNoAllocMinSplits * (size_t)R * (D + 2) > kNoAllocPartFloats) return ESA_ERR_CAPACITY;

    SeqMeta meta;
    int n_att_max = 0;
    for (int b = 0; b < B; ++b) {
        const int64_t t = n_prev[b];
        if (t < 0) return ESA_ERR_INVALID_ARG;
        if (t + l_C > cfg->max_tokens) return ESA_ERR_CAPACITY;
        const int64_t i_end = t < cfg->l_init ? t : cfg->l_init;
        int64_t m_end = t - cfg->l_local;
        if (m_end < i_end) m_end = i_end;
        meta.t[b] = (int)t; meta.i_end[b] = (int)i_end; meta.m_end[b] = (int)m_end;
        const int64_t lM = m_end - i_end;
        const int64_t n = i_end + (lM < cfg->top_k ? lM : cfg->top_k) + (t - m_end) + l_C;
        if (n > n_att_max) n_att_max = (int)n;
    }
    for (int b = B; b < kMaxBatch; ++b) meta.t[b] = meta.i_end[b] = meta.m_end[b] = 0;

    // Once per device, with that device current: resolve the device address of the scratch array
    // (in host code its name is only a handle for the runtime) and read the SM count.
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return ESA_ERR_CUDA;
    if (device < 0 || device >= kNoAllocMaxDevices) return ESA_ERR_UNSUPPORTED;
    std::unique_lock<std::mutex> lock(g_noalloc_mutex);
    NoAllocDevice& dev = g_noalloc_dev[device];
    if (!dev.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_part) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return ESA_ERR_CUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0)
            return ESA_ERR_CUDA;
        dev.part = static_cast<float*>(ptr);
        dev.num_sms = sms;
        dev.ready = true;
    }
    lock.unlock();

    AttendParams p;
    p.Q = (const __nv_bfloat16*)Q_cur; p.K = (const __nv_bfloat16*)K_cache; p.V = (const __nv_bfloat16*)V_cache;
    p.Qg = p.Q; p.Kg = p.K;
    p.O = (__nv_bfloat16*)O; p.idx = idx; p.n_sel = n_sel; p.part = dev.part; p.unit_count = nullptr; p.status = nullptr; p.staged = 0; p.early = 0;
    p.max_tokens = cfg->max_tokens; p.l_C = l_C; p.H = cfg->n_q_heads; p.HG = cfg->n_kv_heads; p.G = G;
    p.top_k = cfg->top_k; p.nsplit = 1;
    const float scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf((float)D);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.meta = meta;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e;
    if (D == 128) e = R <= 16 ? launch_noalloc_t<128, 1, 32>(dev, p, B, n_att_max, st)
                              : launch_noalloc_t<128, 4, 64>(dev, p, B, n_att_max, st);
    else e = R <= 16 ? launch_noalloc_t<64, 1, 32>(dev, p, B, n_att_max, st)
                     : launch_noalloc_t<64, 4, 64>(dev, p, B, n_att_max, st);
    return e == cudaSuccess ? ESA_OK : ESA_ERR_CUDA;
}
