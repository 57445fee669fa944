// Eq. 6 + Eq. 4 (+ Eq. 8) for prefill-sized chunks on the 5th-generation tensor cores.
//
//   S[c, m] = q'_c . k'_m          r_c = max_m S[c, m]          s_m = max_c ( S[c, m] - r_c )
//   s'_j = max of s over [j - eps, j + eps] clipped to M
//
// Two launches stream the compressed keys of the middle tokens through a TMA-fed ring of
// 128-key tiles.  Up to 512 compressed queries of the chunk stay resident in shared memory, so
// a key tile is fetched from L2 once per chunk and pass.  S lives only in tensor memory; the
// accumulator buffers form a ring, so the epilogue of one (tile, query block) item overlaps the
// MMAs of the next:
//   pass 1  queries on the M side (TMEM lanes), keys on the N side, four 128-column buffers: a
//           thread owns one query of each 128-query block and folds the row maximum r_c over
//           every tile in registers.  The items (tile, query block) are dealt out evenly, so
//           CTAs differ by at most one item.  Two warps issue the MMAs of alternate items: a
//           single warp issues one 128x128x16 MMA per ~86 cycles (measured), two reach the tensor
//           core's 64.
//   pass 2  keys on the M side, queries on the N side, two 256-column buffers (a 128x256x16 MMA
//           takes 128 cycles, above one warp's issue time).  The subtraction of r_c rides on the
//           tensor core as a ninth k-step: the key side contributes 1, 1, 1 and the query side the
//           three bf16 pieces of -r_c (r_c = r1 + r2 + r3 exactly), so the accumulator ends as
//           S - r_c -- exactly 0 where S equals r_c bit for bit -- and the epilogue is a plain
//           maximum over the query columns.  (Reading r_c from shared memory in the epilogue
//           instead starves behind the MMAs' operand traffic: measured 2x the MMA time per item.)
//           A CTA owns a contiguous range of keys and also computes the eps keys on either side
//           of it (its tiles start eps keys early and the ranges are 128 n - 2 eps long), so the
//           proximity pooling of Eq. 8 needs no other CTA: pooled scores leave as order-preserving
//           keys, together with the histogram of their top 11 bits (the first radix digit of the
//           selection, Eq. 2).
// Swapping the operands keeps both reductions inside a thread.  Every S[c, m] is the same
// sum of the same exact bf16 products taken in the same order over d' in both passes, so
// pass 2 reproduces pass 1's value and S - r_c is exactly 0 at each query's arg-max.
//
// Chunks of more than 512 queries run as groups of 512 (grid.y); pass 2 then combines the
// groups by an atomic maximum on the unpooled scores and the pooling is left to a later kernel.
//
// Warp roles: warp 0 issues the TMA loads, warps 1-2 issue the MMAs (converged, lane 0 leads;
// pass 2 uses warp 1 only), warps 3-10 run the epilogue: two groups of four warps (one TMEM lane
// quarter each), each group taking one half of an accumulator's columns, with two tensor-memory
// loads in flight per thread.
#include "esa_internal.h"
#include "esa_umma.cuh"

namespace esa {

namespace {

constexpr int ST_KEYS = 128;       // keys per streamed tile
constexpr int ST_THREADS = 352;
constexpr int ST_EPI_WARP0 = 3;    // first epilogue warp
constexpr int ST_EPI = 256;        // epilogue threads
constexpr int ST_QCAP = 512;       // compressed queries resident per CTA
constexpr int ST_BINS = 2048;      // first radix digit: top 11 bits of a key
constexpr int ST_RING = 256;       // pooled-score ring: two tiles of aggregated scores
constexpr int ST_ONES_BYTES = ST_KEYS * 32;    // ninth k-step, key side: 128 rows x 16 bf16
constexpr int ST_RT_BYTES = ST_QCAP * 32;      // ninth k-step, query side: 512 rows x 16 bf16

struct ScoreTcParams {
    uint32_t* rkey;     // [B, l_C] ordered keys of r_c
    uint32_t* skey;     // [B, max_tokens] ordered keys of s_m (index = m - i_end); used when q_groups > 1
    uint32_t* pkey;     // [B, max_tokens] ordered keys of s'_m; written when q_groups == 1
    uint32_t* ghist0;   // [B, ST_BINS] histogram of the top 11 bits of pkey; zeroed by pass 1
    int* status;
    int64_t max_tokens;
    int l_C;
    int eps;
    int q_groups;       // groups of up to ST_QCAP queries (gridDim.y)
    SeqMeta meta;
};

__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;\n" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Operand tiles of the ninth k-step: rows x 16 bf16, K-major without swizzle.  Core matrices of
// 8 rows x 16 bytes are stored as [row group][k half][row][16 B]: the two halves of the k-step
// 128 bytes apart (leading offset), groups of 8 rows 256 bytes apart (stride offset).
__device__ __forceinline__ uint32_t plain_tile_offset(int row, int half) { return (row >> 3) * 256 + half * 128 + (row & 7) * 16; }
__device__ __forceinline__ uint32_t desc_hi_plain() { return (1u << 14) | uint32_t(256 >> 4); }      // descriptor version 1, no swizzle
__device__ __forceinline__ uint32_t desc_lo_plain(uint32_t smem_byte_addr) {
    return ((smem_byte_addr & 0x3ffff) >> 4) | (uint32_t(128 >> 4) << 16);
}

template <int DC, int PASS>
struct ScoreCfg {
    static constexpr int NBLK = DC / 64;                       // 64-column blocks of a row
    static constexpr int UNIT = PASS == 1 ? 128 : 256;         // queries per item
    static constexpr int NBUF = 512 / UNIT;                    // accumulator buffers
    static constexpr int ACC_COLS = PASS == 1 ? ST_KEYS : UNIT;
    static constexpr int STAGES = PASS == 1 ? 3 : 2;
    static constexpr int NMW = PASS == 1 ? 2 : 1;              // warps that issue MMAs
    static constexpr int TILE_BYTES = ST_KEYS * DC * 2;
    static constexpr int Q_BYTES = ST_QCAP * DC * 2;
    static constexpr int EXTRA = PASS == 1 ? 0 : (ST_ONES_BYTES + ST_RT_BYTES + ST_RING * 4 + 2 * ST_KEYS * 4 + ST_BINS * 4);
    static constexpr int SMEM = Q_BYTES + STAGES * TILE_BYTES + EXTRA + 1024;
    static constexpr int MAX_UNITS = ST_QCAP / UNIT;
    // barrier slots
    static constexpr int B_QFULL = 0;
    static constexpr int B_FULL = B_QFULL + MAX_UNITS;
    static constexpr int B_EMPTY = B_FULL + STAGES;
    static constexpr int B_ACC_FULL = B_EMPTY + STAGES;
    static constexpr int B_ACC_EMPTY = B_ACC_FULL + NBUF;
    static constexpr int B_R_READY = B_ACC_EMPTY + NBUF;       // pass 2: the -r_c operand tile is written
    static constexpr int B_COUNT = B_R_READY + 1;
};

template <int DC, int PASS>
__global__ void __launch_bounds__(ST_THREADS, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap qmap, ScoreTcParams p) {
    using C = ScoreCfg<DC, PASS>;
    constexpr int NBLK = C::NBLK, UNIT = C::UNIT, NBUF = C::NBUF, ACC_COLS = C::ACC_COLS, STAGES = C::STAGES, NMW = C::NMW;
    constexpr int TILE_BYTES = C::TILE_BYTES;

    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                                            // [NBLK][ST_QCAP rows][128 B]
    uint8_t* sK = sQ + C::Q_BYTES;                                 // STAGES x [NBLK][128 rows][128 B]
    uint8_t* sOnes = sK + STAGES * TILE_BYTES;                     // pass 2: key side of the ninth k-step
    uint8_t* sRt = sOnes + ST_ONES_BYTES;                          // pass 2: query side of the ninth k-step (pieces of -r_c)
    float* sS = reinterpret_cast<float*>(sRt + ST_RT_BYTES);       // [ST_RING] aggregated scores of the last two tiles
    float* sX = sS + ST_RING;                                      // [2][ST_KEYS] partial maxima of the second column half
    uint32_t* sHist = reinterpret_cast<uint32_t*>(sX + 2 * ST_KEYS);   // [ST_BINS]
    __shared__ uint64_t bars[C::B_COUNT];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int b = blockIdx.z;
    const int q0 = blockIdx.y * ST_QCAP;
    const int nq = min(ST_QCAP, p.l_C - q0);
    const int NU = (nq + UNIT - 1) / UNIT;                 // items per key tile
    const int i_end = p.meta.i_end[b];
    const int l_M = p.meta.m_end[b] - i_end;
    const int eps = p.eps;
    const bool fused = PASS == 2 && p.q_groups == 1;

    // ---- this CTA's keys: local tile lt covers keys [key_first + 128 lt, + 128); its items are
    // w = 0 .. n_items - 1 with (tile, unit) = divmod(w + woff, NU)
    int key_first = 0, n_items = 0, woff = 0, own_lo = 0, own_hi = 0;
    if (l_M > 0) {
        const int n_tiles = (l_M + ST_KEYS - 1) / ST_KEYS;
        if (PASS == 1) {
            const int items = n_tiles * NU;
            const int per = (items + (int)gridDim.x - 1) / (int)gridDim.x;
            const int w0 = min(items, (int)blockIdx.x * per), w1 = min(items, w0 + per);
            key_first = (w0 / NU) * ST_KEYS;
            woff = w0 % NU;
            n_items = w1 - w0;
        } else if (fused) {
            const int share = (l_M + (int)gridDim.x - 1) / (int)gridDim.x;
            const int n = (share + 2 * eps + ST_KEYS - 1) / ST_KEYS;
            const int own = n * ST_KEYS - 2 * eps;           // outputs per CTA
            own_lo = min(l_M, (int)blockIdx.x * own);
            own_hi = min(l_M, own_lo + own);
            if (own_hi > own_lo) {
                key_first = own_lo - eps;
                n_items = ((own_hi - own_lo + 2 * eps + ST_KEYS - 1) / ST_KEYS) * NU;
            }
        } else {
            const int per = (n_tiles + (int)gridDim.x - 1) / (int)gridDim.x;
            const int t0 = min(n_tiles, (int)blockIdx.x * per), t1 = min(n_tiles, t0 + per);
            key_first = t0 * ST_KEYS;
            n_items = (t1 - t0) * NU;
        }
    }
    const int n_ltiles = (n_items + woff + NU - 1) / NU;

    WaitCtx wc{&abort_flag, p.status};
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    if (tid == 0) {
        abort_flag = 0;
        for (int u = 0; u < C::MAX_UNITS; ++u) mbar_init(bar(C::B_QFULL + u), 1);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(C::B_FULL + s), 1);
            mbar_init(bar(C::B_EMPTY + s), NMW);            // one commit per issuing warp and tile
        }
        for (int u = 0; u < NBUF; ++u) {
            mbar_init(bar(C::B_ACC_FULL + u), 1);
            mbar_init(bar(C::B_ACC_EMPTY + u), ST_EPI);
        }
        mbar_init(bar(C::B_R_READY), ST_EPI);
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        // The compressed keys of M were written by launches that completed long ago, and in pass 2 so
        // were the compressed queries (the kernel before the preceding one): those loads go out ahead of
        // the wait for the preceding kernel.  Pass 1 reads queries that the preceding kernel writes.
        if (lane == 0 && n_items > 0) {
            tma_prefetch_desc(&kmap);
            tma_prefetch_desc(&qmap);
            const int64_t row_base = (int64_t)b * p.max_tokens + i_end;
            auto load_tile = [&](int lt) {
                const int s = lt % STAGES;
                mbar_wait(bar(C::B_EMPTY + s), ((lt / STAGES) & 1) ^ 1, wc);
                mbar_arrive_expect_tx(bar(C::B_FULL + s), TILE_BYTES);
#pragma unroll
                for (int blk = 0; blk < NBLK; ++blk)
                    tma_load_2d(smem_u32(sK + s * TILE_BYTES + blk * (ST_KEYS * 128)), &kmap, blk * 64,
                                (int)(row_base + key_first + (int64_t)lt * ST_KEYS), bar(C::B_FULL + s));
            };
            const int first = min(n_ltiles, STAGES);
            for (int lt = 0; lt < first; ++lt) load_tile(lt);
            if (PASS == 1) pdl_wait();
            for (int uu = 0; uu < NU; ++uu) {
                const int u = (uu + woff) % NU;              // in the order the items use them
                mbar_arrive_expect_tx(bar(C::B_QFULL + u), UNIT * DC * 2);
#pragma unroll
                for (int blk = 0; blk < NBLK; ++blk)
#pragma unroll
                    for (int r0 = 0; r0 < UNIT; r0 += 128)
                        tma_load_2d(smem_u32(sQ + blk * (ST_QCAP * 128) + (u * UNIT + r0) * 128), &qmap, blk * 64,
                                    b * p.l_C + q0 + u * UNIT + r0, bar(C::B_QFULL + u));
            }
            for (int lt = first; lt < n_ltiles; ++lt) load_tile(lt);
        }
    } else if (warp <= 2) {
        // ------------------------------------------------------------ MMA issue (converged warps, lane 0 leads)
        // Issuing warp mw takes the items w = mw, mw + NMW, ...  A key stage is released by one commit
        // per issuing warp: each warp commits to the stages of the tiles it has moved past, which covers
        // every MMA it issued on them (and completes at once if it issued none).
        const int mw = warp - 1;
        if (mw < NMW && n_items > 0) {
            const uint32_t lead = lane == 0;
            const uint32_t hi = desc_hi_sw128();
            const uint32_t qlo = desc_lo_kmajor(smem_u32(sQ)), klo = desc_lo_kmajor(smem_u32(sK));
            constexpr uint32_t IDESC = idesc_bf16(128, ACC_COLS, false, false);
            int released = 0;                              // local tiles this warp has released
            int waited = -1;                               // last local tile whose arrival this warp has seen
            for (int w = mw; w < n_items; w += NMW) {
                const int lt = (w + woff) / NU, u = (w + woff) % NU;
                const int s = lt % STAGES, buf = w % NBUF;
                for (; released < lt; ++released) umma_commit(bar(C::B_EMPTY + released % STAGES), lead);
                mbar_wait(bar(C::B_QFULL + u), 0, wc);                       // completes once; later waits pass at once
                if (waited < lt) {
                    mbar_wait(bar(C::B_FULL + s), (lt / STAGES) & 1, wc);
                    waited = lt;
                }
                mbar_wait(bar(C::B_ACC_EMPTY + buf), ((w / NBUF) & 1) ^ 1, wc);
                tc_fence_after_sync();
                const uint32_t k0 = klo + s * (TILE_BYTES >> 4);
                const uint32_t d = tmem + buf * ACC_COLS;
#pragma unroll
                for (int ks = 0; ks < DC / 16; ++ks) {
                    const uint32_t oq = ((ks >> 2) * (ST_QCAP * 128) + u * (UNIT * 128) + (ks & 3) * 32) >> 4;
                    const uint32_t ok = ((ks >> 2) * (ST_KEYS * 128) + (ks & 3) * 32) >> 4;
                    if (PASS == 1) umma_ss(d, qlo + oq, k0 + ok, hi, IDESC, ks, lead);     // S[c, m]
                    else umma_ss(d, k0 + ok, qlo + oq, hi, IDESC, ks, lead);               // S^T[m, c]
                }
                if (PASS == 2) {
                    // ninth k-step: S^T[m, c] += 1 * (-r1) + 1 * (-r2) + 1 * (-r3)
                    mbar_wait(bar(C::B_R_READY), 0, wc);
                    umma_ss(d, desc_lo_plain(smem_u32(sOnes)), desc_lo_plain(smem_u32(sRt + u * (UNIT * 32))), desc_hi_plain(),
                            IDESC, 1, lead);
                }
                umma_commit(bar(C::B_ACC_FULL + buf), lead);
            }
            for (; released < n_ltiles; ++released) umma_commit(bar(C::B_EMPTY + released % STAGES), lead);
        }
    } else {
        // ------------------------------------------------------------ epilogue: 2 groups x 4 warps
        const int quarter = warp & 3;
        const int eg = (warp - ST_EPI_WARP0) >> 2;        // column half of this thread's group
        const int et = quarter * 32 + lane;               // TMEM lane of this thread: 0..127
        const int e256 = eg * 128 + et;
        const uint32_t tbase = tmem_addr(tmem, quarter * 32, 0);
        if (PASS == 2) {
            // key side of the ninth k-step: 1, 1, 1, 0 ... in every row
            if (eg == 0) {
                *reinterpret_cast<uint4*>(sOnes + plain_tile_offset(et, 0)) = make_uint4(0x3f803f80u, 0x00003f80u, 0u, 0u);
                *reinterpret_cast<uint4*>(sOnes + plain_tile_offset(et, 1)) = make_uint4(0u, 0u, 0u, 0u);
            }
            if (fused) {
                for (int i = e256; i < ST_BINS; i += ST_EPI) sHist[i] = 0u;
                for (int i = e256; i < ST_RING; i += ST_EPI) sS[i] = -INFINITY;
            }
        }
        // The next kernel may be set up from here on.  It relies on this order: by the time it starts,
        // every CTA of this grid has seen the preceding grid complete, so whatever that grid and the ones
        // before it wrote is final (which is what lets a kernel load such data ahead of its own wait).
        pdl_wait();
        pdl_launch_dependents();
        if (PASS == 1) {
            // first CTA of a sequence: the histogram that pass 2 (or the pooling kernel) adds to
            if (blockIdx.x == 0 && blockIdx.y == 0)
                for (int i = e256; i < ST_BINS; i += ST_EPI) p.ghist0[(int64_t)b * ST_BINS + i] = 0u;
        } else {
            // query side of the ninth k-step: the three bf16 pieces of -r_c (exact: r_c = r1 + r2 + r3);
            // columns past the chunk get -inf, which no maximum picks
            for (int i = e256; i < ST_QCAP; i += ST_EPI) {
                uint32_t w01 = 0x0000ff80u, w2 = 0u;       // (-inf, 0), (0, 0)
                if (i < nq) {
                    const float r = key_to_f32(p.rkey[(int64_t)b * p.l_C + q0 + i]);
                    const __nv_bfloat16 r1 = __float2bfloat16_rn(r);
                    const float d1 = r - __bfloat162float(r1);
                    const __nv_bfloat16 r2 = __float2bfloat16_rn(d1);
                    const float d2 = d1 - __bfloat162float(r2);
                    const __nv_bfloat16 r3 = __float2bfloat16_rn(d2);
                    w01 = (uint32_t)(__bfloat16_as_ushort(r1) ^ 0x8000u) | ((uint32_t)(__bfloat16_as_ushort(r2) ^ 0x8000u) << 16);
                    w2 = (uint32_t)(__bfloat16_as_ushort(r3) ^ 0x8000u);
                }
                *reinterpret_cast<uint4*>(sRt + plain_tile_offset(i, 0)) = make_uint4(w01, w2, 0u, 0u);
                *reinterpret_cast<uint4*>(sRt + plain_tile_offset(i, 1)) = make_uint4(0u, 0u, 0u, 0u);
            }
            fence_async_smem();
            mbar_arrive(bar(C::B_R_READY));
        }
        float rm0 = -INFINITY, rm1 = -INFINITY, rm2 = -INFINITY, rm3 = -INFINITY;   // pass 1: row maxima per query block
        float a0 = -INFINITY, a1 = -INFINITY, a2 = -INFINITY, a3 = -INFINITY;       // pass 2: running max over the units of a tile
        for (int w = 0; w < n_items; ++w) {
            const int lt = (w + woff) / NU, u = (w + woff) % NU;
            const int buf = w % NBUF;
            const int key0 = key_first + lt * ST_KEYS;
            mbar_wait(bar(C::B_ACC_FULL + buf), (w / NBUF) & 1, wc);
            tc_fence_after_sync();
            if (PASS == 1) {
                // this group's 64 key columns of the item
                const int c0 = eg * 64;
                uint32_t v[64];
                tmem_ld32(tbase + buf * ACC_COLS + c0, v);
                tmem_ld32(tbase + buf * ACC_COLS + c0 + 32, v + 32);
                // (groups of queries: group 0 zeroes the words the groups of pass 2 combine into)
                if (p.q_groups > 1 && blockIdx.y == 0 && eg == 0 && key0 + et < l_M)
                    p.skey[(int64_t)b * p.max_tokens + key0 + et] = 0u;
                tmem_wait_ld();
                tc_fence_before_sync();
                mbar_arrive(bar(C::B_ACC_EMPTY + buf));
                if (key0 + ST_KEYS > l_M) {
#pragma unroll
                    for (int j = 0; j < 64; ++j)
                        if (key0 + c0 + j >= l_M) v[j] = 0xff800000u;
                }
                float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                for (int j = 0; j < 64; j += 8) {
                    m0 = max3f(m0, __uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                    m1 = max3f(m1, __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                    m2 = max3f(m2, __uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
                    m3 = max3f(m3, __uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
                }
                const float rmax = fmaxf(max3f(m0, m1, m2), m3);
                rm0 = u == 0 ? fmaxf(rm0, rmax) : rm0;
                rm1 = u == 1 ? fmaxf(rm1, rmax) : rm1;
                rm2 = u == 2 ? fmaxf(rm2, rmax) : rm2;
                rm3 = u == 3 ? fmaxf(rm3, rmax) : rm3;
            } else {
                if (u == 0) a0 = a1 = a2 = a3 = -INFINITY;
                // this group's 128 query columns of the item, 64 at a time; the accumulator already holds S - r_c
#pragma unroll
                for (int c0 = 0; c0 < 128; c0 += 64) {
                    uint32_t v[64];
                    tmem_ld32(tbase + buf * ACC_COLS + eg * 128 + c0, v);
                    tmem_ld32(tbase + buf * ACC_COLS + eg * 128 + c0 + 32, v + 32);
                    tmem_wait_ld();
                    if (c0 == 64) {
                        tc_fence_before_sync();
                        mbar_arrive(bar(C::B_ACC_EMPTY + buf));
                    }
#pragma unroll
                    for (int j = 0; j < 64; j += 8) {
                        a0 = max3f(a0, __uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                        a1 = max3f(a1, __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                        a2 = max3f(a2, __uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
                        a3 = max3f(a3, __uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
                    }
                }
                if (u == NU - 1) {
                    // the two column halves meet: group 1 hands its partial maximum to group 0
                    float sm = fmaxf(max3f(a0, a1, a2), a3);
                    if (eg == 1) sX[(lt & 1) * ST_KEYS + et] = sm;
                    asm volatile("bar.sync 2, 256;\n" ::: "memory");
                    if (eg == 0) {
                        sm = fmaxf(sm, sX[(lt & 1) * ST_KEYS + et]);
                        const int m = key0 + et;                                  // this thread's key
                        if (!fused) {
                            if (m < l_M) atomicMax(p.skey + (int64_t)b * p.max_tokens + m, f32_to_key(sm));
                        } else {
                            // Eq. 8: keys outside M never win a window; outputs lag the scores by eps keys
                            sS[(lt * ST_KEYS + et) & (ST_RING - 1)] = (m >= 0 && m < l_M) ? sm : -INFINITY;
                            asm volatile("bar.sync 1, 128;\n" ::: "memory");
                            const int ul = lt * ST_KEYS - eps + et;               // local index of this thread's output
                            const int mo = key_first + ul;
                            const bool valid = ul >= eps && mo >= own_lo && mo < own_hi;
                            float best = -INFINITY;
                            if (valid)
                                for (int dlt = -eps; dlt <= eps; ++dlt) best = fmaxf(best, sS[(ul + dlt) & (ST_RING - 1)]);
                            const uint32_t key = f32_to_key(best);
                            if (valid) p.pkey[(int64_t)b * p.max_tokens + mo] = key;
                            // histogram of the first radix digit, aggregated over the warp (neighbouring keys crowd into few bins)
                            const uint32_t peers = __match_any_sync(0xffffffffu, valid ? (key >> 21) : 0xffffffffu);
                            if (valid && lane == __ffs(peers) - 1) atomicAdd(&sHist[key >> 21], (uint32_t)__popc(peers));
                            asm volatile("bar.sync 1, 128;\n" ::: "memory");      // the ring slot of tile lt - 1 may be overwritten next
                        }
                    }
                }
            }
        }
        if (PASS == 1) {
            const int qb = q0 + et;
            uint32_t* rk = p.rkey + (int64_t)b * p.l_C;
            if (qb < p.l_C && rm0 > -INFINITY) atomicMax(rk + qb, f32_to_key(rm0));
            if (qb + 128 < p.l_C && rm1 > -INFINITY) atomicMax(rk + qb + 128, f32_to_key(rm1));
            if (qb + 256 < p.l_C && rm2 > -INFINITY) atomicMax(rk + qb + 256, f32_to_key(rm2));
            if (qb + 384 < p.l_C && rm3 > -INFINITY) atomicMax(rk + qb + 384, f32_to_key(rm3));
        } else if (fused && n_items > 0) {
            asm volatile("bar.sync 2, 256;\n" ::: "memory");
            uint32_t* gh = p.ghist0 + (int64_t)b * ST_BINS;
            for (int i = e256; i < ST_BINS; i += ST_EPI) {
                const uint32_t c = sHist[i];
                if (c) atomicAdd(gh + i, c);
            }
        }
    }
    // (every thread passes the wait for the preceding kernel before the CTA ends: a CTA's exit also
    // releases the dependents, and they must not start ahead of the kernels before this one)
    pdl_wait();

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

template <int DC>
cudaError_t launch_t(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache, const SeqMeta& meta, int max_lM,
                     cudaStream_t st, bool* pooled_ready) {
    CUtensorMap kmap, qmap;
    if (!make_tensor_map_bf16(&kmap, kc_cache, (uint64_t)B * ctx->cfg.max_tokens, DC, 128)) return cudaErrorNotSupported;
    if (!make_tensor_map_bf16(&qmap, ctx->Qc, (uint64_t)B * l_C, DC, 128)) return cudaErrorNotSupported;
    ScoreTcParams p;
    p.rkey = ctx->rkey; p.skey = ctx->skey; p.pkey = ctx->pkey; p.ghist0 = ctx->ghist0; p.status = ctx->status;
    p.max_tokens = ctx->cfg.max_tokens; p.l_C = l_C; p.eps = ctx->cfg.eps; p.meta = meta;
    const int q_groups = (l_C + ST_QCAP - 1) / ST_QCAP;
    p.q_groups = q_groups;
    using C1 = ScoreCfg<DC, 1>;
    using C2 = ScoreCfg<DC, 2>;
    cudaError_t e = cudaFuncSetAttribute(score_tc_kernel<DC, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, C1::SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_tc_kernel<DC, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, C2::SMEM);
    if (e != cudaSuccess) return e;
    const int n_tiles = (max_lM + ST_KEYS - 1) / ST_KEYS;
    int per_seq = ctx->num_sms / (q_groups * B);
    if (per_seq < 1) per_seq = 1;
    // pass 1: items of 128 queries x 128 keys
    const int nq = l_C < ST_QCAP ? l_C : ST_QCAP;
    int gx1 = per_seq;
    const int items1 = n_tiles * ((nq + 127) / 128);
    if (gx1 > items1) gx1 = items1;
    if (gx1 < 1) gx1 = 1;
    {
        ProfScope prof(ctx, KC_SCORE_PASS1, st);
        e = launch_pdl(score_tc_kernel<DC, 1>, dim3(gx1, q_groups, B), dim3(ST_THREADS), C1::SMEM, st, kmap, qmap, p);
    }
    if (e != cudaSuccess) return e;
    // pass 2: whole tiles (every query of a group) per CTA
    int gx2 = per_seq;
    if (gx2 > n_tiles) gx2 = n_tiles;
    if (gx2 < 1) gx2 = 1;
    {
        ProfScope prof(ctx, KC_SCORE_PASS2, st);
        e = launch_pdl(score_tc_kernel<DC, 2>, dim3(gx2, q_groups, B), dim3(ST_THREADS), C2::SMEM, st, kmap, qmap, p);
    }
    if (e != cudaSuccess) return e;
    ctx->launches += 2;
    *pooled_ready = q_groups == 1;
    return cudaGetLastError();
}

}  // namespace

// Both scoring passes for chunks of at least 64 queries and d' of 64 or 128; rkey must be zeroed.
// *pooled_ready: ctx->pkey and ctx->ghist0 hold the pooled keys and their first-digit histogram
// (else ctx->skey holds the unpooled keys and ghist0 is zero).
// Returns cudaErrorNotSupported when this path does not cover the shape.
cudaError_t launch_score_tc(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache, const SeqMeta& meta,
                            int max_lM, cudaStream_t st, bool* pooled_ready) {
    if (l_C < 64) return cudaErrorNotSupported;
    if (ctx->dc == 128) return launch_t<128>(ctx, B, l_C, kc_cache, meta, max_lM, st, pooled_ready);
    if (ctx->dc == 64) return launch_t<64>(ctx, B, l_C, kc_cache, meta, max_lM, st, pooled_ready);
    return cudaErrorNotSupported;
}

}  // namespace esa
