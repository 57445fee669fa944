// Eq. 6 + Eq. 4 (+ Eq. 8) for prefill-sized chunks on the 5th-generation tensor cores.
//
//   S[c, m] = q'_c . k'_m          r_c = max_m S[c, m]          s_m = max_c ( S[c, m] - r_c )
//   s'_j = max of s over [j - eps, j + eps] clipped to M
//
// Two launches stream the compressed keys of the middle tokens through a TMA-fed ring of
// 128-key tiles.  Up to 512 compressed queries of the chunk stay resident in shared memory, so
// a key tile is fetched from L2 once per chunk and pass and feeds 2048 tensor-core cycles.  S
// lives only in tensor memory; the accumulator buffers form a ring, so the epilogue of one
// (tile, query block) item overlaps the MMAs of the next:
//   pass 1  queries on the M side (TMEM lanes), keys on the N side, four 128-column buffers: a
//           thread owns one query of each 128-query block and folds the row maximum r_c over
//           every tile in registers.  The items (tile, query block) are dealt out evenly, so
//           CTAs differ by at most one 512-cycle item.
//   pass 2  keys on the M side, queries on the N side, two 256-column buffers: a thread owns
//           one key, subtracts the r_c of every query column and keeps the maximum over all
//           queries of the chunk.  A CTA owns a contiguous range of keys and also computes the
//           eps keys on either side of it (its tiles start eps keys early and the ranges are
//           128 n - 2 eps long), so the proximity pooling of Eq. 8 needs no other CTA: pooled
//           scores leave as order-preserving keys, together with the histogram of their top 11
//           bits (the first radix digit of the selection, Eq. 2).
// Swapping the operands keeps both reductions inside a thread.  Every S[c, m] is the same
// sum of the same exact bf16 products taken in the same order over d' in both passes, so
// pass 2 reproduces pass 1's value and S - r_c is exactly 0 at each query's arg-max.
//
// Chunks of more than 512 queries run as groups of 512 (grid.y); pass 2 then combines the
// groups by an atomic maximum on the unpooled scores and the pooling is left to a later kernel.
//
// Warp roles: warp 0 issues the TMA loads, warp 1 issues the MMAs (converged, lane 0
// leads), warps 2-5 run the epilogue (one TMEM lane quarter each).
#include "esa_internal.h"
#include "esa_umma.cuh"

namespace esa {

namespace {

constexpr int ST_KEYS = 128;       // keys per streamed tile
constexpr int ST_THREADS = 192;
constexpr int ST_QCAP = 512;       // compressed queries resident per CTA
constexpr int ST_BINS = 2048;      // first radix digit: top 11 bits of a key
constexpr int ST_RING = 256;       // pooled-score ring: two tiles of aggregated scores

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

template <int DC, int PASS>
struct ScoreCfg {
    static constexpr int NBLK = DC / 64;                       // 64-column blocks of a row
    static constexpr int UNIT = PASS == 1 ? 128 : 256;         // queries per item
    static constexpr int NBUF = 512 / UNIT;                    // accumulator buffers (UNIT columns each in pass 2, 128 in pass 1)
    static constexpr int ACC_COLS = PASS == 1 ? ST_KEYS : UNIT;
    static constexpr int STAGES = PASS == 1 ? 3 : 2;
    static constexpr int TILE_BYTES = ST_KEYS * DC * 2;
    static constexpr int Q_BYTES = ST_QCAP * DC * 2;
    static constexpr int EXTRA = PASS == 1 ? 0 : (ST_QCAP * 4 + ST_RING * 4 + ST_BINS * 4);
    static constexpr int SMEM = Q_BYTES + STAGES * TILE_BYTES + EXTRA + 1024;
    static constexpr int MAX_UNITS = ST_QCAP / UNIT;
    // barrier slots
    static constexpr int B_QFULL = 0;
    static constexpr int B_FULL = B_QFULL + MAX_UNITS;
    static constexpr int B_EMPTY = B_FULL + STAGES;
    static constexpr int B_ACC_FULL = B_EMPTY + STAGES;
    static constexpr int B_ACC_EMPTY = B_ACC_FULL + NBUF;
    static constexpr int B_COUNT = B_ACC_EMPTY + NBUF;
};

template <int DC, int PASS>
__global__ void __launch_bounds__(ST_THREADS, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap qmap, ScoreTcParams p) {
    using C = ScoreCfg<DC, PASS>;
    constexpr int NBLK = C::NBLK, UNIT = C::UNIT, NBUF = C::NBUF, ACC_COLS = C::ACC_COLS, STAGES = C::STAGES;
    constexpr int TILE_BYTES = C::TILE_BYTES;

    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                                            // [NBLK][ST_QCAP rows][128 B]
    uint8_t* sK = sQ + C::Q_BYTES;                                 // STAGES x [NBLK][128 rows][128 B]
    float* sR = reinterpret_cast<float*>(sK + STAGES * TILE_BYTES);    // [ST_QCAP] r_c (pass 2)
    float* sS = sR + ST_QCAP;                                      // [ST_RING] aggregated scores of the last two tiles
    uint32_t* sHist = reinterpret_cast<uint32_t*>(sS + ST_RING);   // [ST_BINS]
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
            mbar_init(bar(C::B_EMPTY + s), 1);
        }
        for (int u = 0; u < NBUF; ++u) {
            mbar_init(bar(C::B_ACC_FULL + u), 1);
            mbar_init(bar(C::B_ACC_EMPTY + u), 128);
        }
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    pdl_wait();
    pdl_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
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
            // the first key tile goes out before the queries: the first MMA needs both
            load_tile(0);
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
            for (int lt = 1; lt < n_ltiles; ++lt) load_tile(lt);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issue (converged warp, lane 0 leads)
        if (n_items > 0) {
            const uint32_t lead = lane == 0;
            const uint32_t hi = desc_hi_sw128();
            const uint32_t qlo = desc_lo_kmajor(smem_u32(sQ)), klo = desc_lo_kmajor(smem_u32(sK));
            constexpr uint32_t IDESC = idesc_bf16(128, ACC_COLS, false, false);
            for (int w = 0; w < n_items; ++w) {
                const int lt = (w + woff) / NU, u = (w + woff) % NU;
                const int s = lt % STAGES, buf = w % NBUF;
                mbar_wait(bar(C::B_QFULL + u), 0, wc);                       // completes once; later waits pass at once
                if (w == 0 || u == 0) mbar_wait(bar(C::B_FULL + s), (lt / STAGES) & 1, wc);
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
                if (u == NU - 1 || w == n_items - 1) umma_commit(bar(C::B_EMPTY + s), lead);
                umma_commit(bar(C::B_ACC_FULL + buf), lead);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue: 4 warps, one TMEM lane quarter each
        const int quarter = warp & 3;
        const int et = quarter * 32 + lane;               // TMEM lane of this thread: 0..127
        const uint32_t tbase = tmem_addr(tmem, quarter * 32, 0);
        if (PASS == 1) {
            // first CTA of a sequence: the histogram that pass 2 (or the pooling kernel) adds to
            if (blockIdx.x == 0 && blockIdx.y == 0)
                for (int i = et; i < ST_BINS; i += 128) p.ghist0[(int64_t)b * ST_BINS + i] = 0u;
        } else {
            for (int i = et; i < ST_QCAP; i += 128)
                sR[i] = (i < nq) ? key_to_f32(p.rkey[(int64_t)b * p.l_C + q0 + i]) : INFINITY;
            if (fused) {
                for (int i = et; i < ST_BINS; i += 128) sHist[i] = 0u;
                for (int i = et; i < ST_RING; i += 128) sS[i] = -INFINITY;
            }
            asm volatile("bar.sync 1, 128;\n" ::: "memory");
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
                const bool tail = key0 + ST_KEYS > l_M;
                // (groups of queries: group 0 zeroes the words the groups of pass 2 combine into)
                if (p.q_groups > 1 && blockIdx.y == 0 && key0 + et < l_M) p.skey[(int64_t)b * p.max_tokens + key0 + et] = 0u;
                float rmax = -INFINITY;
#pragma unroll
                for (int c0 = 0; c0 < ST_KEYS; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tbase + buf * ACC_COLS + c0, v);
                    tmem_wait_ld();
                    if (tail) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (key0 + c0 + j >= l_M) v[j] = 0xff800000u;
                    }
                    float m0 = rmax, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        m0 = max3f(m0, __uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                        m1 = max3f(m1, __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                        m2 = max3f(m2, __uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
                        m3 = max3f(m3, __uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
                    }
                    rmax = fmaxf(max3f(m0, m1, m2), m3);
                }
                tc_fence_before_sync();
                mbar_arrive(bar(C::B_ACC_EMPTY + buf));
                rm0 = u == 0 ? fmaxf(rm0, rmax) : rm0;
                rm1 = u == 1 ? fmaxf(rm1, rmax) : rm1;
                rm2 = u == 2 ? fmaxf(rm2, rmax) : rm2;
                rm3 = u == 3 ? fmaxf(rm3, rmax) : rm3;
            } else {
                if (u == 0) a0 = a1 = a2 = a3 = -INFINITY;
                const float* rr = sR + u * UNIT;
#pragma unroll
                for (int c0 = 0; c0 < UNIT; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tbase + buf * ACC_COLS + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        const float4 ra = *reinterpret_cast<const float4*>(rr + c0 + j);
                        const float4 rb = *reinterpret_cast<const float4*>(rr + c0 + j + 4);
                        a0 = max3f(a0, __uint_as_float(v[j]) - ra.x, __uint_as_float(v[j + 1]) - ra.y);
                        a1 = max3f(a1, __uint_as_float(v[j + 2]) - ra.z, __uint_as_float(v[j + 3]) - ra.w);
                        a2 = max3f(a2, __uint_as_float(v[j + 4]) - rb.x, __uint_as_float(v[j + 5]) - rb.y);
                        a3 = max3f(a3, __uint_as_float(v[j + 6]) - rb.z, __uint_as_float(v[j + 7]) - rb.w);
                    }
                }
                tc_fence_before_sync();
                mbar_arrive(bar(C::B_ACC_EMPTY + buf));
                if (u == NU - 1) {
                    const float sm = fmaxf(max3f(a0, a1, a2), a3);
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
        if (PASS == 1) {
            const int qb = q0 + et;
            uint32_t* rk = p.rkey + (int64_t)b * p.l_C;
            if (qb < p.l_C && rm0 > -INFINITY) atomicMax(rk + qb, f32_to_key(rm0));
            if (qb + 128 < p.l_C && rm1 > -INFINITY) atomicMax(rk + qb + 128, f32_to_key(rm1));
            if (qb + 256 < p.l_C && rm2 > -INFINITY) atomicMax(rk + qb + 256, f32_to_key(rm2));
            if (qb + 384 < p.l_C && rm3 > -INFINITY) atomicMax(rk + qb + 384, f32_to_key(rm3));
        } else if (fused && n_items > 0) {
            uint32_t* gh = p.ghist0 + (int64_t)b * ST_BINS;
            for (int i = et; i < ST_BINS; i += 128) {
                const uint32_t c = sHist[i];
                if (c) atomicAdd(gh + i, c);
            }
        }
    }

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
