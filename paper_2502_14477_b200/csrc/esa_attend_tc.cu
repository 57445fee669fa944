// Eq. 1 / Algorithm 1 for prefill-sized chunks on the 5th-generation tensor cores.
//
// Same computation as the split kernel in esa_attend.cu (one softmax over the key list
// I u M_k u L u C, C causal), organised for tcgen05:
//
//   * A CTA owns 256 rows (row = query c * G + head-in-group g) of one key/value head: two
//     128-row Q tiles that share every K/V tile brought into shared memory.
//   * Scores S = Q K^T and outputs O += P V accumulate in tensor memory: per Q tile 128
//     columns of S and D columns of O (512 columns in all).  P (bf16) overwrites the first
//     half of its own S columns and is read by the second MMA straight from tensor memory.
//   * Warp roles: warps 0-3 / 4-7 run the online softmax of Q tile 0 / 1 (one thread per
//     row holding its 128 scores in registers, so row maxima and row sums need no shuffles)
//     and warps 8-11 gather K/V rows with index-driven 16-byte cp.async into
//     128-byte-swizzled tiles.  The MMAs of a Q tile are issued by one thread of its own
//     softmax warpgroup, right after the group has stored P: a separate issuing warp is
//     starved of issue slots by the arithmetic-heavy softmax warps it shares a scheduler with
//     (measured: 100-600 cycles per tcgen05.mma instead of 64).  While one Q tile is in its
//     softmax the tensor core works on the other.
//   * Half of the exponentials are evaluated on the FMA pipe (Cody-Waite split + cubic), the
//     rest on the special-function unit, whose 16 results per clock would otherwise bound
//     the kernel at about half the tensor rate.
//   * The running maximum is only raised when it grows by more than 2^8: until then the
//     exponentials are taken against the stale maximum (bounded by 256, exact in fp32/bf16
//     range), which makes rescaling O in tensor memory rare; (O, m, l) stay consistent, so
//     the final division, or the split merge, needs no correction.
//   * A long key list can be split across CTAs (blockIdx.z); partial (O, m, l) go to the
//     context's scratch and the merge kernel of esa_attend.cu combines them.
#include "esa_internal.h"
#include "esa_umma.cuh"

namespace esa {

namespace {

constexpr int TC_BN = 128;            // keys per tile
constexpr int TC_ROWS = 256;          // rows per CTA
constexpr int TC_SOFTMAX_WARPS = 8;
constexpr int TC_PRODUCER_WARPS = 4;
constexpr int TC_THREADS = (TC_SOFTMAX_WARPS + TC_PRODUCER_WARPS) * 32;
// Register split after start-up.  setmaxnreg.inc draws from the pool the CTA was launched with
// and blocks until the pool can serve it, so the split must fit that pool exactly:
// launch = 384 threads x 168 registers; 8 warps x 208 + 4 warps x 88 = the same 2016 per lane.
constexpr int TC_REGS_LAUNCH = 168;
constexpr int TC_REGS_SOFTMAX = 208;
constexpr int TC_REGS_OTHER = 88;
static_assert(TC_SOFTMAX_WARPS * TC_REGS_SOFTMAX + TC_PRODUCER_WARPS * TC_REGS_OTHER <=
                  (TC_SOFTMAX_WARPS + TC_PRODUCER_WARPS) * TC_REGS_LAUNCH,
              "register split exceeds the CTA's launch allocation: setmaxnreg.inc would never return");
constexpr int TC_POLY_PAIRS_OF_4 = 2; // of every 4 column pairs, this many take 2^x on the FMA pipe
constexpr int TC_PRODUCERS = TC_PRODUCER_WARPS * 32;
constexpr float kRescaleThreshold = 8.0f;    // log2 domain

struct TcAttendParams {
    const __nv_bfloat16* Q;
    const __nv_bfloat16* K;
    const __nv_bfloat16* V;
    __nv_bfloat16* O;
    const int32_t* idx;
    const int32_t* n_sel;
    float* part;
    int* status;
    int64_t max_tokens;
    int l_C, H, HG, G, top_k;
    int nsplit;
    float scale_log2;
    SeqMeta meta;
};

// barrier slots in shared memory
enum {
    BAR_Q_FULL = 0,
    BAR_K_FULL = 1,    // 2
    BAR_V_FULL = 3,    // 2
    BAR_K_EMPTY = 5,   // 2
    BAR_V_EMPTY = 7,   // 2
    BAR_S_READY = 9,   // 2 (per Q tile)
    BAR_O_READY = 11,  // 2
    BAR_COUNT = 13
};

__device__ __forceinline__ void cp_async_arrive_noinc(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(bar) : "memory");
}
template <int N>
__device__ __forceinline__ void reg_alloc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void reg_dealloc() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(N));
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;\n" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// two-wide fp32 arithmetic (one instruction for a pair of columns)
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{\n.reg .b64 ra, rb, rc, rd;\nmov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %5};\nmov.b64 rc, {%6, %7};\n"
        "fma.rn.f32x2 rd, ra, rb, rc;\nmov.b64 {%0, %1}, rd;\n}\n"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    float2 d;
    asm("{\n.reg .b64 ra, rb, rd;\nmov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %5};\n"
        "add.rn.f32x2 rd, ra, rb;\nmov.b64 {%0, %1}, rd;\n}\n"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
// 2^x for a pair, x <= ~10, on the FMA pipe: x = n + f with n = round(x), f in [-0.5, 0.5];
// 2^f by a degree-3 minimax polynomial (relative error 7.5e-5, far below the bf16 rounding
// of P), n added into the exponent field.  x is clamped at -126 (result ~ 1e-38).
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
    const float kMagic = 12582912.0f;                       // 1.5 * 2^23: low mantissa bits hold round(x)
    x.x = fmaxf(x.x, -126.0f);
    x.y = fmaxf(x.y, -126.0f);
    const float2 t = fadd2(x, make_float2(kMagic, kMagic));
    const float2 n = fadd2(t, make_float2(-kMagic, -kMagic));
    const float2 f = ffma2(n, make_float2(-1.f, -1.f), x);
    float2 q = ffma2(f, make_float2(0.0551716685f, 0.0551716685f), make_float2(0.242611125f, 0.242611125f));
    q = ffma2(q, f, make_float2(0.693260968f, 0.693260968f));
    q = ffma2(q, f, make_float2(0.999928057f, 0.999928057f));
    float2 r;
    r.x = __uint_as_float(__float_as_uint(q.x) + (__float_as_uint(t.x) << 23));
    r.y = __uint_as_float(__float_as_uint(q.y) + (__float_as_uint(t.y) << 23));
    return r;
}

template <int D>
__global__ void __launch_bounds__(TC_THREADS, 1)
attend_tc_kernel(TcAttendParams p) {
    constexpr int CH = D / 8;                  // 16-byte chunks per row
    constexpr int TILE_BYTES = TC_BN * D * 2;  // one K or V tile, also one Q tile
    constexpr int BLK_BYTES = 128 * 128;       // one 64-column block of a 128-row tile

    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                           // 2 Q tiles
    uint8_t* sK = sQ + 2 * TILE_BYTES;            // 2 stages
    uint8_t* sV = sK + 2 * TILE_BYTES;            // 2 stages
    __shared__ uint64_t bars[BAR_COUNT];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row0 = blockIdx.x * TC_ROWS;
    const int kvh = blockIdx.y;
    const int b = blockIdx.z / p.nsplit;
    const int split = blockIdx.z % p.nsplit;
    const int G = p.G;
    const int R = p.l_C * G;

    const int t = p.meta.t[b], i_end = p.meta.i_end[b], m_end = p.meta.m_end[b];
    int n_sel = p.n_sel[b];
    n_sel = max(0, min(n_sel, min(p.top_k, m_end - i_end)));
    const int n_glob = i_end + n_sel;
    const int n_att = n_glob + (t - m_end) + p.l_C;
    const int c_first = n_att - p.l_C;

    const int r_last = min(R, row0 + TC_ROWS) - 1;
    const int j_end = c_first + r_last / G + 1;           // keys visible to the last row of the CTA
    const int n_tiles_all = (j_end + TC_BN - 1) / TC_BN;
    const int per = (n_tiles_all + p.nsplit - 1) / p.nsplit;
    const int tile_begin = split * per;
    const int tile_end = min(n_tiles_all, tile_begin + per);
    const int n_tiles = max(0, tile_end - tile_begin);

    WaitCtx wc{&abort_flag, p.status};
    auto bar = [&](int i) { return smem_u32(&bars[i]); };

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar(BAR_Q_FULL), TC_PRODUCERS);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(BAR_K_FULL + s), TC_PRODUCERS);
            mbar_init(bar(BAR_V_FULL + s), TC_PRODUCERS);
            mbar_init(bar(BAR_K_EMPTY + s), 2);      // one commit per Q tile
            mbar_init(bar(BAR_V_EMPTY + s), 2);
            mbar_init(bar(BAR_S_READY + s), 1);
            mbar_init(bar(BAR_O_READY + s), 1);
        }
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    // columns: S of Q tile q at q * 128, O of Q tile q at 256 + q * D
    if (warp < TC_SOFTMAX_WARPS) reg_alloc<TC_REGS_SOFTMAX>();
    else reg_dealloc<TC_REGS_OTHER>();

    if (warp < TC_SOFTMAX_WARPS) {
        // ------------------------------------------------------------ softmax, one row per thread
        const int qt = warp >> 2;                        // Q tile of this warpgroup
        const int lane_base = (warp & 3) * 32;           // TMEM lanes this warp may touch
        const int row = row0 + qt * 128 + lane_base + lane;
        const uint32_t tS = tmem_addr(tmem, lane_base, qt * 128);
        const uint32_t tO = tmem_addr(tmem, lane_base, 256 + qt * D);
        const int lim = c_first + min(row / G, p.l_C - 1) + 1;          // first invisible list position
        const int lim_min = c_first + min((row0 + qt * 128) / G, p.l_C - 1) + 1;   // smallest limit of the tile
        const float sl2 = p.scale_log2;
        float m_run = -INFINITY, l_run = 0.f;

        // ---- MMA issue: lane 0 of the group's first warp
        const bool issuer = (warp & 3) == 0 && lane == 0;
        constexpr uint32_t ID_QK = idesc_bf16(128, TC_BN, false, false);
        constexpr uint32_t ID_PV = idesc_bf16(128, D, false, true);
        const uint32_t hi = desc_hi_sw128();
        const uint32_t qlo = desc_lo_kmajor(smem_u32(sQ)) + qt * (TILE_BYTES >> 4);
        const uint32_t klo = desc_lo_kmajor(smem_u32(sK)), vlo = desc_lo_mnmajor(smem_u32(sV), BLK_BYTES);
        const uint32_t dS = tmem + qt * 128, dO = tmem + 256 + qt * D;
        // descriptor low words advance by compile-time constants (bytes >> 4)
        auto issue_qk = [&](int s) {
            const uint32_t b0 = klo + s * (TILE_BYTES >> 4);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const uint32_t o = ((ks >> 2) * BLK_BYTES + (ks & 3) * 32) >> 4;
                umma_ss(dS, qlo + o, b0 + o, hi, ID_QK, ks);
            }
        };
        auto issue_pv = [&](int s, int acc) {
            const uint32_t b0 = vlo + s * (TILE_BYTES >> 4);
#pragma unroll
            for (int ks = 0; ks < TC_BN / 16; ++ks) umma_ts(dO, dS + ks * 8, b0 + ks * (2048 >> 4), hi, ID_PV, acc | ks);
        };
        if (issuer && n_tiles > 0) {
            mbar_wait(bar(BAR_Q_FULL), 0, wc);
            mbar_wait(bar(BAR_K_FULL + 0), 0, wc);
            fence_async_smem();
            tc_fence_after_sync();
            issue_qk(0);
            umma_commit(bar(BAR_S_READY + qt));
            umma_commit(bar(BAR_K_EMPTY + 0));
        }
        __syncwarp();

        for (int j = 0; j < n_tiles; ++j) {
            const int key0 = (tile_begin + j) * TC_BN;
            mbar_wait(bar(BAR_S_READY + qt), j & 1, wc);
            tc_fence_after_sync();
            const bool need_mask = key0 + TC_BN > lim_min;
            // the whole score row of this thread: 128 fp32 columns
            uint32_t v[TC_BN];
#pragma unroll
            for (int c0 = 0; c0 < TC_BN; c0 += 32) tmem_ld32(tS + c0, v + c0);
            tmem_wait_ld();
            if (need_mask) {
#pragma unroll
                for (int i = 0; i < TC_BN; ++i)
                    if (key0 + i >= lim) v[i] = 0xff800000u;     // -inf
            }
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int i = 0; i < TC_BN; i += 4) {
                mx0 = fmax3(mx0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                mx1 = fmax3(mx1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
            }
            const float m_new = fmaxf(m_run, fmaxf(mx0, mx1) * sl2);
            const bool grow = m_new > m_run + kRescaleThreshold;
            if (__any_sync(0xffffffffu, grow)) {
                // 0 on a row's first visible tile; a row that has seen no key yet keeps (m, l) = (-inf, 0)
                const float alpha = (m_new == -INFINITY) ? 1.f : fast_exp2(m_run - m_new);
                l_run *= alpha;
                m_run = m_new;
                if (j > 0) {
                    // the commit that made S ready also covers the previous P V product: O is quiescent
#pragma unroll
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        uint32_t o[32];
                        tmem_ld32(tO + c0, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(tO + c0, o);
                    }
                }
            }
            // P = 2^(S * scale - m) as packed bf16 over the first half of the S columns.
            // A row without a visible key so far has m = -inf: its P must be 0, not 2^(+inf).
            const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
            const float2 sl2v = make_float2(sl2, sl2), nm = make_float2(neg_m, neg_m);
            float2 sum2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int c0 = 0; c0 < TC_BN; c0 += 32) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float2 x = ffma2(make_float2(__uint_as_float(v[c0 + 2 * i]), __uint_as_float(v[c0 + 2 * i + 1])),
                                           sl2v, nm);
                    float2 e;
                    if ((i & 3) < TC_POLY_PAIRS_OF_4) {
                        e = exp2_poly2(x);
                    } else {
                        e.x = fast_exp2(x.x);
                        e.y = fast_exp2(x.y);
                    }
                    sum2 = fadd2(sum2, e);
                    pk[i] = pack_bf16(e.x, e.y);
                }
                tmem_st16(tS + (c0 >> 1), pk);
            }
            l_run += sum2.x + sum2.y;
            tmem_wait_st();
            tc_fence_before_sync();
            // every row of P is in tensor memory: named barrier over the 128 threads of the group
            asm volatile("bar.sync %0, 128;\n" ::"r"(1 + qt) : "memory");
            if (issuer) {
                const int s = j & 1, sn = s ^ 1;
                tc_fence_after_sync();
                mbar_wait(bar(BAR_V_FULL + s), (j >> 1) & 1, wc);
                fence_async_smem();
                issue_pv(s, j > 0);
                umma_commit(bar(BAR_V_EMPTY + s));
                if (j + 1 < n_tiles) {
                    mbar_wait(bar(BAR_K_FULL + sn), ((j + 1) >> 1) & 1, wc);
                    fence_async_smem();
                    issue_qk(sn);                      // overwrites S (and P) after the P V product, in issue order
                    umma_commit(bar(BAR_S_READY + qt));
                    umma_commit(bar(BAR_K_EMPTY + sn));
                } else {
                    umma_commit(bar(BAR_O_READY + qt));
                }
            }
            __syncwarp();
        }

        // ---- epilogue: O / l  (or the unnormalised partial for the split merge)
        if (n_tiles > 0) {
            mbar_wait(bar(BAR_O_READY + qt), 0, wc);
            tc_fence_after_sync();
        }
        const bool row_ok = row < R;
        const int cq = row_ok ? row / G : 0, g = row_ok ? row % G : 0;
        if (p.nsplit == 1) {
            const float inv = 1.f / l_run;
            __nv_bfloat16* dst = p.O + (((int64_t)b * p.l_C + cq) * p.H + kvh * G + g) * D;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tO + c0, v);
                tmem_wait_ld();
                if (row_ok) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(v[q4 * 8 + 0]) * inv, __uint_as_float(v[q4 * 8 + 1]) * inv);
                        o.y = pack_bf16(__uint_as_float(v[q4 * 8 + 2]) * inv, __uint_as_float(v[q4 * 8 + 3]) * inv);
                        o.z = pack_bf16(__uint_as_float(v[q4 * 8 + 4]) * inv, __uint_as_float(v[q4 * 8 + 5]) * inv);
                        o.w = pack_bf16(__uint_as_float(v[q4 * 8 + 6]) * inv, __uint_as_float(v[q4 * 8 + 7]) * inv);
                        *reinterpret_cast<uint4*>(dst + c0 + q4 * 8) = o;
                    }
                }
            }
        } else {
            float* dst = p.part + ((((int64_t)b * p.HG + kvh) * p.nsplit + split) * R + (row_ok ? row : 0)) * (D + 2);
            if (n_tiles > 0) {
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tO + c0, v);
                    tmem_wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 32; i += 2)
                            *reinterpret_cast<float2*>(dst + c0 + i) =
                                make_float2(__uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                    }
                }
            }
            if (row_ok) {
                dst[D] = m_run;        // -inf marks an empty part
                dst[D + 1] = l_run;
            }
        }
    } else {
        // ------------------------------------------------------------ producers: Q, then K/V tiles
        const int ptid = tid - TC_SOFTMAX_WARPS * 32;      // 0..127
        const int chunk = ptid % CH;                       // this thread's 16-byte chunk of every row
        const int rsub = ptid / CH;                        // first row handled
        constexpr int RSTEP = TC_PRODUCERS / CH;           // rows advanced per iteration
        const uint32_t blk_off = (chunk >> 3) * BLK_BYTES; // 64-column block of the chunk
        const int cin = chunk & 7;
        if (n_tiles > 0) {
            for (int r = rsub; r < TC_ROWS; r += RSTEP) {
                const int row = row0 + r;
                const bool ok = row < R;
                const int cq = ok ? row / G : 0, g = ok ? row % G : 0;
                const __nv_bfloat16* src = p.Q + (((int64_t)b * p.l_C + cq) * p.H + kvh * G + g) * D + chunk * 8;
                const int rr = r & 127;
                uint8_t* dst = sQ + (r >> 7) * TILE_BYTES + blk_off + rr * 128 + ((cin ^ (rr & 7)) << 4);
                cp_async16(dst, src, ok ? 16 : 0);
            }
            cp_async_arrive_noinc(bar(BAR_Q_FULL));
        }
        const __nv_bfloat16* Kb = p.K + ((int64_t)b * p.max_tokens * p.HG + kvh) * D + chunk * 8;
        const __nv_bfloat16* Vb = p.V + ((int64_t)b * p.max_tokens * p.HG + kvh) * D + chunk * 8;
        const int32_t* idx = p.idx + (int64_t)b * p.top_k;
        const int64_t tok_stride = (int64_t)p.HG * D;
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j & 1;
            const uint32_t ph = ((j >> 1) & 1) ^ 1;
            const int key0 = (tile_begin + j) * TC_BN;
            // positions of this thread's rows
            int pos[TC_BN / RSTEP];
#pragma unroll
            for (int it = 0; it < TC_BN / RSTEP; ++it) {
                const int jj = key0 + rsub + it * RSTEP;
                int q = -1;
                if (jj < i_end) q = jj;
                else if (jj < n_glob) q = __ldg(idx + (jj - i_end));
                else if (jj < n_att) q = m_end + (jj - n_glob);
                pos[it] = q;
            }
            mbar_wait(bar(BAR_K_EMPTY + s), ph, wc);
#pragma unroll
            for (int it = 0; it < TC_BN / RSTEP; ++it) {
                const int r = rsub + it * RSTEP;
                uint8_t* dst = sK + s * TILE_BYTES + blk_off + r * 128 + ((cin ^ (r & 7)) << 4);
                cp_async16(dst, Kb + (pos[it] < 0 ? 0 : pos[it]) * tok_stride, pos[it] < 0 ? 0 : 16);
            }
            cp_async_arrive_noinc(bar(BAR_K_FULL + s));
            mbar_wait(bar(BAR_V_EMPTY + s), ph, wc);
#pragma unroll
            for (int it = 0; it < TC_BN / RSTEP; ++it) {
                const int r = rsub + it * RSTEP;
                uint8_t* dst = sV + s * TILE_BYTES + blk_off + r * 128 + ((cin ^ (r & 7)) << 4);
                cp_async16(dst, Vb + (pos[it] < 0 ? 0 : pos[it]) * tok_stride, pos[it] < 0 ? 0 : 16);
            }
            cp_async_arrive_noinc(bar(BAR_V_FULL + s));
        }
        cp_async_wait<0>();
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

}  // namespace

template <int D>
static cudaError_t launch_tc(esa_ctx* ctx, TcAttendParams& p, int B, int n_att_max, cudaStream_t st, int* nsplit_out) {
    const int R = p.l_C * p.G;
    const int row_tiles = (R + TC_ROWS - 1) / TC_ROWS;
    constexpr int smem = 6 * TC_BN * D * 2 + 1024;
    cudaError_t e = cudaFuncSetAttribute(attend_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    // the in-kernel register split assumes the launch allocation it was sized for
    static int regs_checked = 0;
    if (!regs_checked) {
        cudaFuncAttributes fa;
        e = cudaFuncGetAttributes(&fa, attend_tc_kernel<D>);
        if (e != cudaSuccess) return e;
        if (fa.numRegs != TC_REGS_LAUNCH) return cudaErrorInvalidConfiguration;
        regs_checked = 1;
    }
    // Split the key list when that fills the machine better: cost model = waves x tiles per CTA
    // (+1 tile-equivalent of fixed work per CTA), one CTA per SM.
    const int ctas = row_tiles * p.HG * B;
    const int n_tiles = (n_att_max + TC_BN - 1) / TC_BN;
    int best = 1;
    double best_cost = 1e30;
    for (int ns = 1; ns <= kAttPrefillSplits && ns <= n_tiles; ++ns) {
        if ((size_t)B * p.HG * ns * R * (D + 2) > ctx->att_part_elems) break;
        const int per = (n_tiles + ns - 1) / ns;
        const int waves = (ctas * ns + ctx->num_sms - 1) / ctx->num_sms;
        const double cost = (double)waves * (per + 1.0) + (ns > 1 ? 0.5 * ns : 0.0);
        if (cost < best_cost - 1e-9) { best_cost = cost; best = ns; }
    }
    p.nsplit = best;
    *nsplit_out = best;
    attend_tc_kernel<D><<<dim3(row_tiles, p.HG, B * best), TC_THREADS, smem, st>>>(p);
    ctx->launches += 1;
    return cudaGetLastError();
}

// Returns cudaErrorNotSupported when this path does not cover the shape (the caller then
// uses the split kernel); nsplit_out tells the caller whether a merge pass must follow.
cudaError_t launch_attend_tc(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                             const __nv_bfloat16* V, const SeqMeta& meta, const int32_t* idx, const int32_t* n_sel,
                             __nv_bfloat16* O, int n_att_max, cudaStream_t st, int* nsplit_out) {
    TcAttendParams p;
    p.Q = Q; p.K = K; p.V = V; p.O = O; p.idx = idx; p.n_sel = n_sel; p.part = ctx->att_part; p.status = ctx->status;
    p.max_tokens = ctx->cfg.max_tokens; p.l_C = l_C; p.H = ctx->H; p.HG = ctx->HG; p.G = ctx->G;
    p.top_k = ctx->cfg.top_k; p.nsplit = 1;
    p.scale_log2 = ctx->scale * 1.4426950408889634f;
    p.meta = meta;
    if (ctx->d == 128) return launch_tc<128>(ctx, p, B, n_att_max, st, nsplit_out);
    if (ctx->d == 64) return launch_tc<64>(ctx, p, B, n_att_max, st, nsplit_out);
    return cudaErrorNotSupported;
}

}  // namespace esa
