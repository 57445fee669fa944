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
// scores and accumulators.  Small chunks (decode) split the key list across CTAs and a
// second kernel merges the partial (O, m, l) triples -- the same algebra as Algorithm 1's
// merge.
#include "esa_internal.h"

namespace esa {

struct AttendParams {
    const __nv_bfloat16* Q;   // [B, l_C, H, D]
    const __nv_bfloat16* K;   // [B, max_tokens, HG, D]
    const __nv_bfloat16* V;
    __nv_bfloat16* O;         // [B, l_C, H, D]
    const int32_t* idx;       // [B, top_k]
    const int32_t* n_sel;     // [B]
    float* part;              // split partials
    int64_t max_tokens;
    int l_C, H, HG, G, top_k;
    int nsplit;
    float scale_log2;         // softmax scale * log2(e)
    SeqMeta meta;
};

// layout of the split-KV partial buffer, per (b, kvh, split): R rows x (D + 2) floats
// (unnormalised O row, running max m in the exp2 domain, running sum l)

template <int D, int NW, int BN>
__global__ void __launch_bounds__(NW * 32)
attend_kernel(AttendParams p) {
    constexpr int CH = D / 8;
    constexpr int BM = NW * 16;
    constexpr int NT = NW * 32;
    extern __shared__ uint4 smem[];
    uint4* sQ = smem;                         // [BM][CH]
    uint4* sK = sQ + BM * CH;                 // 2 x [BN][CH]
    uint4* sV = sK + 2 * BN * CH;             // 2 x [BN][CH]

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
    const __nv_bfloat16* Vb = p.V + ((int64_t)b * p.max_tokens * p.HG + kvh) * D;
    const int32_t* idx = p.idx + (int64_t)b * p.top_k;
    const int64_t tok_stride = (int64_t)p.HG * D;

    auto load_kv = [&](int st, int tile) {
        uint4* dk = sK + st * BN * CH;
        uint4* dv = sV + st * BN * CH;
        for (int i = tid; i < BN * CH; i += NT) {
            int r = i / CH, c = i % CH;
            int j = tile * BN + r;
            bool ok = j < n_att;
            int pos = 0;
            if (ok) {
                if (j < i_end) pos = j;
                else if (j < n_glob) pos = __ldg(idx + (j - i_end));
                else pos = m_end + (j - n_glob);
            }
            const int64_t off = (int64_t)pos * tok_stride + c * 8;
            cp_async16(&dk[swz<CH>(r, c)], Kb + off, ok ? 16 : 0);
            cp_async16(&dv[swz<CH>(r, c)], Vb + off, ok ? 16 : 0);
        }
    };

    // Q tile -> smem (rows past R are zero)
    for (int i = tid; i < BM * CH; i += NT) {
        int r = i / CH, c = i % CH;
        int row = row0 + r;
        bool ok = row < R;
        int cq = ok ? row / G : 0, g = ok ? row % G : 0;
        const __nv_bfloat16* src = p.Q + (((int64_t)b * p.l_C + cq) * p.H + kvh * G + g) * D + c * 8;
        cp_async16(&sQ[swz<CH>(r, c)], src, ok ? 16 : 0);
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

        // scale, mask (causal inside C and the ragged tail), online softmax
        const int j0 = tile * BN;
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
template <int D>
__global__ void __launch_bounds__(256) attend_merge_kernel(AttendParams p) {
    constexpr int PER = D / 32;                  // columns per lane: 2 or 4
    const int R = p.l_C * p.G;
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int kvh = blockIdx.y, b = blockIdx.z;
    if (row >= R) return;
    const float* base = p.part + (((int64_t)b * p.HG + kvh) * p.nsplit * R + row) * (D + 2);
    const int64_t sstride = (int64_t)R * (D + 2);
    float M = -INFINITY;
    for (int s = 0; s < p.nsplit; ++s) M = fmaxf(M, __ldg(base + s * sstride + D));
    float den = 0.f;
    float acc[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) acc[i] = 0.f;
    for (int s = 0; s < p.nsplit; ++s) {
        const float* ps = base + s * sstride;
        const float m = __ldg(ps + D);
        if (m == -INFINITY) continue;            // an empty part (uniform over the warp)
        const float w = fast_exp2(m - M);
        den += w * __ldg(ps + D + 1);
        // rows start at multiples of (D + 2) floats: 8-byte aligned, so read pairs
#pragma unroll
        for (int i = 0; i < PER; i += 2) {
            const float2 v = __ldg(reinterpret_cast<const float2*>(ps + lane * PER + i));
            acc[i] += w * v.x;
            acc[i + 1] += w * v.y;
        }
    }
    const float inv = 1.f / den;
    const int cq = row / p.G, g = row % p.G;
    __nv_bfloat16* dst = p.O + (((int64_t)b * p.l_C + cq) * p.H + kvh * p.G + g) * D + lane * PER;
#pragma unroll
    for (int i = 0; i < PER; i += 2) *reinterpret_cast<uint32_t*>(dst + i) = pack_bf16(acc[i] * inv, acc[i + 1] * inv);
}

template <int D, int NW, int BN>
static cudaError_t launch_attend_t(esa_ctx* ctx, AttendParams& p, int B, int n_att_max, cudaStream_t st) {
    constexpr int BM = NW * 16;
    const int R = p.l_C * p.G;
    const int row_tiles = (R + BM - 1) / BM;
    constexpr int smem = (BM + 4 * BN) * (D / 8) * 16;
    cudaError_t e = cudaFuncSetAttribute(attend_kernel<D, NW, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int nsplit = 1;
    if (R <= kAttSplitRows && row_tiles == 1) {
        // split the key list so that one wave of CTAs fills the machine (never a second, short wave)
        int per_sm = 1;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attend_kernel<D, NW, BN>, NW * 32, smem);
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
    attend_kernel<D, NW, BN><<<dim3(row_tiles, p.HG, B * nsplit), NW * 32, smem, st>>>(p);
    ctx->launches += 1;
    if (nsplit > 1) {
        attend_merge_kernel<D><<<dim3((R + 7) / 8, p.HG, B), 256, 0, st>>>(p);
        ctx->launches += 1;
    }
    return cudaGetLastError();
}

cudaError_t launch_attend(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                          const __nv_bfloat16* V, const SeqMeta& meta, const int32_t* idx,
                          const int32_t* n_sel, __nv_bfloat16* O, cudaStream_t st) {
    AttendParams p;
    p.Q = Q; p.K = K; p.V = V; p.O = O; p.idx = idx; p.n_sel = n_sel; p.part = ctx->att_part;
    p.max_tokens = ctx->cfg.max_tokens; p.l_C = l_C; p.H = ctx->H; p.HG = ctx->HG; p.G = ctx->G;
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
        // prefill-sized chunks: tcgen05 kernel, then the merge when it split the key list
        int nsplit = 1;
        cudaError_t e = launch_attend_tc(ctx, B, l_C, Q, K, V, meta, idx, n_sel, O, n_att_max, st, &nsplit);
        if (e != cudaSuccess) return e;
        if (nsplit > 1) {
            p.nsplit = nsplit;
            if (ctx->d == 128) attend_merge_kernel<128><<<dim3((R + 7) / 8, p.HG, B), 256, 0, st>>>(p);
            else attend_merge_kernel<64><<<dim3((R + 7) / 8, p.HG, B), 256, 0, st>>>(p);
            ctx->launches += 1;
        }
        return cudaGetLastError();
    }
    if (ctx->d == 128) {
        if (R <= 16) return launch_attend_t<128, 1, 32>(ctx, p, B, n_att_max, st);
        if (R <= 64) return launch_attend_t<128, 4, 64>(ctx, p, B, n_att_max, st);
        return launch_attend_t<128, 8, 64>(ctx, p, B, n_att_max, st);
    } else if (ctx->d == 64) {
        if (R <= 16) return launch_attend_t<64, 1, 32>(ctx, p, B, n_att_max, st);
        if (R <= 64) return launch_attend_t<64, 4, 64>(ctx, p, B, n_att_max, st);
        return launch_attend_t<64, 8, 64>(ctx, p, B, n_att_max, st);
    }
    return cudaErrorInvalidValue;
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

template <int D, int NW, int BN>
cudaError_t launch_noalloc_t(const NoAllocDevice& dev, AttendParams& p, int B, int n_att_max, cudaStream_t st) {
    const int R = p.l_C * p.G;
    constexpr int smem = (NW * 16 + 4 * BN) * (D / 8) * 16;
    cudaError_t e = cudaFuncSetAttribute(attend_kernel<D, NW, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int per_sm = 1;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attend_kernel<D, NW, BN>, NW * 32, smem);
    if (e != cudaSuccess) return e;
    const int n_tiles = (n_att_max + BN - 1) / BN;
    int nsplit = (per_sm * dev.num_sms) / (p.HG * B);
    if (nsplit > kAttMaxSplits) nsplit = kAttMaxSplits;
    if (nsplit > n_tiles) nsplit = n_tiles;
    while (nsplit > 1 && (size_t)B * p.HG * nsplit * R * (D + 2) > kNoAllocPartFloats) --nsplit;
    if (nsplit < 1) nsplit = 1;
    p.nsplit = nsplit;
    attend_kernel<D, NW, BN><<<dim3(1, p.HG, B * nsplit), NW * 32, smem, st>>>(p);
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

    AttendParams p;
    p.Q = (const __nv_bfloat16*)Q_cur; p.K = (const __nv_bfloat16*)K_cache; p.V = (const __nv_bfloat16*)V_cache;
    p.O = (__nv_bfloat16*)O; p.idx = idx; p.n_sel = n_sel; p.part = dev.part;
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
