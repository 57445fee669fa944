// Eq. 1 / Algorithm 1 for prefill-sized chunks on the 5th-generation tensor cores.
//
// Same computation as the split kernel in esa_attend.cu (one softmax over the key list
// I u M_k u L u C, C causal), organised for tcgen05:
//
//   * A CTA owns 256 rows (row = query c * G + head-in-group g) of one key/value head: two
//     128-row Q tiles that share every 128-key K/V tile brought into shared memory.
//   * Scores S = Q K^T and outputs O += P V accumulate in tensor memory.  Per Q tile: 128 columns
//     of S (one 128-key tile, written by products of N = 128: an instruction of N = 64 occupies the
//     tensor pipe as long as one of N = 128, measured, and with 64-key tiles that pipe bounded the loop)
//     and D columns of O, 512 columns in all.  The softmax handles a tile as two 64-key halves: P (bf16)
//     of a half overwrites the first 32 columns of that half and is read by the second MMA straight from
//     tensor memory, so P V of the first half runs while the exponentials of the second are being taken.
//   * Per Q tile the chain is S ready -> softmax (two halves) -> P V, then Q K^T of the next tile into
//     the same columns (the tensor core executes one thread's products in issue order).  One warp issues
//     for both Q tiles in a fixed alternating order, which keeps them half a period apart: the tensor
//     core works for one while the other is in its softmax.
//   * Warp roles: warps 0-3 / 4-7 run the online softmax of Q tile 0 / 1 (one thread per
//     row holding the 64 scores of a half in registers, so row sums need no shuffles),
//     warps 8-11 gather K/V rows with index-driven 16-byte cp.async into 128-byte-swizzled
//     tiles, warp 12 issues the MMAs.  It runs converged (all lanes compute
//     the warp-uniform descriptors, lane 0 executes the tcgen05 instructions): a single
//     diverged thread was starved of issue slots by the arithmetic-heavy softmax warps that
//     share its scheduler (measured 100-600 cycles per tcgen05.mma instead of 64).
//   * Every exponential is one ex2.approx on the special-function unit.  (Evaluating a share of them on the
//     FMA pipe -- Cody-Waite split + cubic -- was measured at 1/16, 1/8, 1/4, 3/8 and 1/2 of the scores, with
//     64-key and with 128-key tiles, and was slower than none at every share.)
//   * The running maximum m is set on a row's first tile and after that only raised when a half's sum of
//     2^(score - m) reaches 2^64: the exponentials are taken against m as it stands, with no search for the
//     half's maximum first and hardly ever a rescaling of O in tensor memory; (O, m, l) stay consistent
//     whatever m is, so the final division, or the split merge, needs no correction, and fp32 (sums, O) and
//     bf16 (P) carry the range.
//   * A long key list can be split across CTAs (blockIdx.z); a two-way split runs as CTA pairs that exchange
//     halves of their partial (O, m, l) through distributed shared memory (PAIR, below); otherwise the partials
//     go to the context's scratch through coalesced stores, and the CTA that finishes a unit last merges
//     them with its own accumulator (an arrival counter per unit decides; nobody waits).
//   * A call that follows the selection of its step (p.early) takes the attended set as two lists: I then L,
//     whose rows are older than the chunk and do not depend on the selection, before the kernel's wait for the
//     preceding kernel, and M_k then C after it.  Every role runs the two phases in turn; the selection kernel
//     (a handful of busy SMs) runs beside the first.  The issuing warp takes the wait at the start of the last
//     early tile's round; one issuing warp it stays (two, sharing the k-steps of every product, were slower
//     whether they alternated strictly or ran freely, and the free-running pair gave up the fixed order of sums).
//   * Two-position attention (Section 3.2) is a split by construction: the first half of the splits
//     covers the list entries of I and M_k with the second encoding (Qg, Kg), the other half covers
//     L and C with (Q, K), so a CTA holds one pair of Q tiles whichever part it works on, and the
//     merge that joins key-list splits also joins the two parts (Algorithm 1's merge of (O, m, l)).
#include <cstring>

#include "esa_internal.h"
#include "esa_umma.cuh"

namespace esa {

namespace {

constexpr int TC_BN = 128;            // keys per tile
constexpr int TC_HALF = 64;           // keys per softmax step (half a tile)
constexpr int TC_ROWS = 256;          // rows per CTA
constexpr int TC_STAGES = 2;          // K tiles and V tiles in shared memory
constexpr int TC_SOFTMAX_WARPS = 8;
constexpr int TC_PRODUCER_WARPS = 4;
constexpr int TC_MMA_WARP = TC_SOFTMAX_WARPS + TC_PRODUCER_WARPS;
constexpr int TC_THREADS = 512;       // 13 working warps, padded to whole warpgroups for setmaxnreg
constexpr int TC_PRODUCERS = TC_PRODUCER_WARPS * 32;
// Register split after start-up.  setmaxnreg.inc draws from the pool the CTA was launched with
// and blocks until the pool can serve it, so the split must fit that pool:
// launch = 16 warps x 128 registers; 8 warps x 168 + 8 warps x 88 = the same 2048 per lane.
constexpr int TC_REGS_LAUNCH = 128;
constexpr int TC_REGS_SOFTMAX = 168;
constexpr int TC_REGS_OTHER = 88;
static_assert(kAttPrefillSplits == 4, "the in-kernel merge selects among four weights");
static_assert(8 * TC_REGS_SOFTMAX + 8 * TC_REGS_OTHER <= 16 * TC_REGS_LAUNCH,
              "register split exceeds the CTA's launch allocation: setmaxnreg.inc would never return");
constexpr float kSumLimit = 1.8446744e19f;   // 2^64: a tile whose sum of 2^(score - m) reaches this has its maximum looked up

struct TcAttendParams {
    const __nv_bfloat16* Q;
    const __nv_bfloat16* K;
    const __nv_bfloat16* Qg;   // two-position attention (Section 3.2): queries / keys used against I and M_k
    const __nv_bfloat16* Kg;
    const __nv_bfloat16* V;
    __nv_bfloat16* O;
    const int32_t* idx;
    const int32_t* n_sel;
    float* part;
    int* status;
    int64_t max_tokens;
    int l_C, H, HG, G, top_k;
    int nsplit;
    int Rp;             // rows of a scratch part (R rounded up to even: 16-byte aligned parts)
    int* unit_count;    // arrivals per (sequence, key/value head, row tile); returns to 0 after each launch
    int q_tma;          // Q tiles arrive by TMA (one arrival) instead of cp.async (one per producer thread)
    int staged;         // the caches hold the attended list itself: row j = list entry j
    int early;          // the rows of I and L are attended ahead of the wait for the preceding kernel (never with staged or two)
    int two;            // two-position attention: splits [0, nsplit/2) take I and M_k with (Qg, Kg), the rest L and C with (Q, K)
    float scale_log2;
    SeqMeta meta;
};

// barrier slots in shared memory
enum {
    BAR_Q_FULL = 0,
    BAR_K_FULL = 1,                         // TC_STAGES
    BAR_V_FULL = BAR_K_FULL + TC_STAGES,    // TC_STAGES
    BAR_K_EMPTY = BAR_V_FULL + TC_STAGES,   // TC_STAGES
    BAR_V_EMPTY = BAR_K_EMPTY + TC_STAGES,  // TC_STAGES
    BAR_S_READY = BAR_V_EMPTY + TC_STAGES,  // per Q tile: 2, one phase per tile
    BAR_P_READY = BAR_S_READY + 2,          // [Q tile][half]: 4, one phase per tile
    BAR_PV_DONE = BAR_P_READY + 4,          // per Q tile: 2, one phase per half
    BAR_O_READY = BAR_PV_DONE + 2,          // per Q tile: 2, completes once
    BAR_PAIR = BAR_O_READY + 2,             // PAIR: the partner's half of the partial result has landed; completes once
    BAR_COUNT = BAR_PAIR + 1
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
// Barrier over all threads of a thread-block cluster, split in two so that warps with nothing to publish
// can arrive early.  Arrive releases this thread's shared-memory writes, wait acquires the others'.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;\n" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;\n" ::: "memory"); }
// address of the same shared-memory location in another CTA of the cluster
__device__ __forceinline__ uint32_t cluster_map(uint32_t smem_addr, uint32_t cta_rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(smem_addr), "r"(cta_rank));
    return r;
}
// Bulk copy from this CTA's shared memory into another CTA's of the cluster; the bytes are counted on the
// destination CTA's mbarrier.  Addresses and size are multiples of 16.
__device__ __forceinline__ void bulk_copy_to_cluster(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes, uint32_t mbar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst_cluster),
                 "r"(src_cta), "r"(bytes), "r"(mbar_cluster)
                 : "memory");
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
// The merged rows of one column half (DH columns) leave as bf16 through a per-warp staging buffer: 16-byte
// stores, whole rows per instruction.  acc: this lane's row; lane rr of the warp owns row wrow0 + rr, whose
// element offset in O is (own_hi : own_lo).
template <int DH>
__device__ __forceinline__ void store_half_rows(const float* acc, float4* stage, int lane, int wrow0, int R, uint32_t own_lo,
                                                uint32_t own_hi, __nv_bfloat16* O_half) {
    constexpr int NB = DH / 8;               // uint4 per staged row
    uint4* st16 = reinterpret_cast<uint4*>(stage);
#pragma unroll
    for (int q8 = 0; q8 < NB; ++q8) {
        uint4 o4;
        o4.x = pack_bf16(acc[q8 * 8 + 0], acc[q8 * 8 + 1]);
        o4.y = pack_bf16(acc[q8 * 8 + 2], acc[q8 * 8 + 3]);
        o4.z = pack_bf16(acc[q8 * 8 + 4], acc[q8 * 8 + 5]);
        o4.w = pack_bf16(acc[q8 * 8 + 6], acc[q8 * 8 + 7]);
        st16[lane * NB + (q8 ^ (lane & (NB - 1)))] = o4;
    }
    __syncwarp();
#pragma unroll
    for (int it = 0; it < NB; ++it) {
        const int e = it * 32 + lane, rr = e / NB, c = e % NB;
        const uint32_t lo = __shfl_sync(0xffffffffu, own_lo, rr), hi32 = __shfl_sync(0xffffffffu, own_hi, rr);
        if (wrow0 + rr < R) {
            __nv_bfloat16* d2 = O_half + (((int64_t)hi32 << 32) | lo);
            *reinterpret_cast<uint4*>(d2 + c * 8) = st16[rr * NB + (c ^ (rr & (NB - 1)))];
        }
    }
    __syncwarp();
}

// PAIR: the key list is split in two and the two CTAs of a unit form a thread-block cluster.  CTA r finishes
// column half r of the unit's rows.  Each parks the other column half of its partial (O, m, l) in its own shared
// memory (the K/V stages, idle by then); after a cluster barrier (both CTAs have finished their products) each
// sends that half into the partner's shared memory with bulk copies counted on the partner's mbarrier, and once
// its own mbarrier has counted the incoming bytes it merges the received half with its accumulator in tensor
// memory and writes the bf16 rows: no round trip through global memory, no fences, no arrival counter.
// (Measured for the 128 KB of a partial: loads from the other CTA's shared memory 9 us, one 16-byte store per
// lane and row 6 us, bulk copies 3.5 us.)  A second cluster barrier keeps each sender's shared memory alive until
// its copies have landed.
template <int D, bool PAIR>
__global__ void __launch_bounds__(TC_THREADS, 1)
attend_tc_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap qgmap, TcAttendParams p) {
    constexpr int STAGES = TC_STAGES;
    constexpr int CH = D / 8;                   // 16-byte chunks per row
    constexpr int Q_TILE_BYTES = 128 * D * 2;   // one 128-row Q tile
    constexpr int Q_BLK_BYTES = 128 * 128;      // one 64-column block of it
    constexpr int KV_TILE_BYTES = TC_BN * D * 2;
    constexpr int KV_BLK_BYTES = TC_BN * 128;

    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                               // 2 Q tiles
    uint8_t* sK = sQ + 2 * Q_TILE_BYTES;              // STAGES tiles
    uint8_t* sV = sK + STAGES * KV_TILE_BYTES;        // STAGES tiles
    __shared__ uint64_t bars[BAR_COUNT];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int merge_ticket;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int warp_u = __shfl_sync(0xffffffffu, warp, 0);     // provably warp-uniform copy
    const int row0 = blockIdx.x * TC_ROWS;
    const int kvh = blockIdx.y;
    const int b = blockIdx.z / p.nsplit;
    const int split = blockIdx.z % p.nsplit;
    const int G = p.G;
    const int R = p.l_C * G;

    WaitCtx wc{&abort_flag, p.status};
    auto bar = [&](int i) { return smem_u32(&bars[i]); };

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar(BAR_Q_FULL), p.q_tma ? 1 : TC_PRODUCERS);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(BAR_K_FULL + s), TC_PRODUCERS);
            mbar_init(bar(BAR_V_FULL + s), TC_PRODUCERS);
            mbar_init(bar(BAR_K_EMPTY + s), 1);          // one commit, after the products of both Q tiles
            mbar_init(bar(BAR_V_EMPTY + s), 1);
        }
        for (int s = 0; s < 4; ++s) mbar_init(bar(BAR_P_READY + s), 128);   // every softmax thread of the Q tile arrives
        for (int q = 0; q < 2; ++q) {
            mbar_init(bar(BAR_S_READY + q), 1);
            mbar_init(bar(BAR_PV_DONE + q), 1);
            mbar_init(bar(BAR_O_READY + q), 1);
        }
        mbar_init(bar(BAR_PAIR), 1);
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    // columns: S of Q tile q at q * 128 (half u at + u * 64); O of Q tile q at 256 + q * D
    // The rows of I and L are older than the chunk and depend on nothing the preceding kernels of the step write (the
    // selection least of all).  With `p.early` the attended set is taken as two lists: the early one, I then L, whose
    // tiles every CTA shares out and attends BEFORE its wait for the preceding kernel (the selection kernel is then
    // still at work on a handful of SMs), and the late one, the selected entries then C, attended after the wait.
    // Otherwise (two position encodings, caches that hold the staged list, or a call that does not follow the
    // selection of its step) there is one list, I, M_k, L, C, and all of it comes after the wait.
    // A list is described by four numbers: entry j is cache row j below `ie`, idx[j - ie] below `ng`, cache row
    // me + (j - ng) from there on, and nothing from `row_lim` on.
    struct KeyList { int ie, ng, me, row_lim; };
    const int t = p.meta.t[b], i_end = p.meta.i_end[b], m_end = p.meta.m_end[b];
    const int r_last = min(R, row0 + TC_ROWS) - 1;
    const int e_len = p.early ? i_end + (t - m_end) : 0;                 // entries of the early list
    const int early_all = (e_len + TC_BN - 1) / TC_BN;
    const int early_per = (early_all + p.nsplit - 1) / p.nsplit;
    const int early_begin = min(early_all, split * early_per);
    const int n_early = min(early_all, early_begin + early_per) - early_begin;      // this CTA's early tiles
    const KeyList list_early = {i_end, i_end, m_end, e_len};
    // set after the wait: the late (or only) list, this CTA's part of it, and the tile count of both phases
    KeyList list_late = {0, 0, 0, 0};
    int c_first = 0, part_lo = 0, part_hi = 0, tile_begin = 0, n_tiles = 0;
    bool far = false, planned = false;
    auto plan = [&]() {
        pdl_wait();
        pdl_launch_dependents();
        int n_sel = p.n_sel[b];
        n_sel = max(0, min(n_sel, min(p.top_k, m_end - i_end)));
        if (p.early) list_late = {0, n_sel, t, n_sel + p.l_C};
        else list_late = {i_end, i_end + n_sel, m_end, i_end + n_sel + (t - m_end) + p.l_C};
        c_first = list_late.row_lim - p.l_C;                  // entry of the chunk's first token
        const int j_end = c_first + r_last / G + 1;           // keys visible to the last row of the CTA
        // The part of the key list this CTA's group of splits covers: all of it, or (two-position attention)
        // the entries of I and M_k for the first half of the splits and those of L and C for the second.
        const int grp = p.two ? p.nsplit / 2 : p.nsplit;       // splits that share a part
        far = p.two && split < grp;                            // this CTA works with (Qg, Kg)
        part_lo = (p.two && !far) ? list_late.ng : 0;
        part_hi = far ? list_late.ng : j_end;
        if (far) list_late.row_lim = part_hi;
        // (with an early list the shares run the other way round: the split with the short early share comes first)
        const int s_in = (p.two && !far) ? split - grp : (p.early ? grp - 1 - split : split);
        const int late_all = max(0, (part_hi - part_lo + TC_BN - 1) / TC_BN);
        if (p.early && grp == 2 && late_all >= 2) {
            // Two splits: the late list is cut where the first split's early and late tiles together make half of
            // all tiles (rounded up).  The second split, which holds the masked tiles of C (the dearer ones), is then
            // never the one with a tile more.
            const int cut = min(late_all, max(0, ((early_all + late_all + 1) >> 1) - min(early_all, early_per)));
            tile_begin = split == 0 ? 0 : cut;
            n_tiles = n_early + (split == 0 ? cut : late_all - cut);
        } else {
            const int per = (late_all + grp - 1) / grp;
            tile_begin = min(late_all, s_in * per);
            n_tiles = n_early + min(late_all, tile_begin + per) - tile_begin;
        }
        planned = true;
    };
    if (n_early == 0) plan();
    // Every role takes its tiles in two phases, the early ones and, after `plan`, the late ones; tile j of the CTA
    // starts at entry key_first + (j - j_first) * TC_BN of the phase's list.
    const bool has_work = n_early > 0 || n_tiles > 0;

    if (warp_u < TC_SOFTMAX_WARPS) reg_alloc<TC_REGS_SOFTMAX>();
    else reg_dealloc<TC_REGS_OTHER>();

    if (warp_u < TC_SOFTMAX_WARPS) {
        // ------------------------------------------------------------ softmax, one row per thread
        const int qt = warp_u >> 2;                      // Q tile of this warpgroup
        const int lane_base = (warp_u & 3) * 32;         // TMEM lanes this warp may touch
        const int row = row0 + qt * 128 + lane_base + lane;
        const uint32_t tS = tmem_addr(tmem, lane_base, qt * 128);
        const uint32_t tO = tmem_addr(tmem, lane_base, 256 + qt * D);
        const float sl2 = p.scale_log2;
        float m_run = -INFINITY, l_run = 0.f;

#pragma unroll 1
        for (int phase = 0; phase < 2; ++phase) {
        if (phase == 1 && !planned) plan();
        const int j_first = phase == 0 ? 0 : 2 * n_early, j_last = phase == 0 ? 2 * n_early : 2 * n_tiles;
        const int key_first = phase == 0 ? early_begin * TC_BN : part_lo + tile_begin * TC_BN;
        // first invisible entry of this row, and the smallest such limit of the Q tile (every row sees all of the
        // early list)
        const int lim = phase == 0 ? e_len : min(part_hi, c_first + min(row / G, p.l_C - 1) + 1);
        const int lim_min = phase == 0 ? e_len : min(part_hi, c_first + min((row0 + qt * 128) / G, p.l_C - 1) + 1);
        for (int j = j_first; j < j_last; ++j) {            // j counts halves: tile j >> 1, half j & 1
            const int T = j >> 1, u = j & 1;
            const int key0 = key_first + (j - j_first) * TC_HALF;
            if (u == 0) {
                mbar_wait(bar(BAR_S_READY + qt), T & 1, wc);
                tc_fence_after_sync();
            }
            const bool need_mask = key0 + TC_HALF > lim_min;
            // the score row of this thread: 64 fp32 columns
            uint32_t v[TC_HALF];
            tmem_ld32(tS + u * 64, v);
            tmem_ld32(tS + u * 64 + 32, v + 32);
            tmem_wait_ld();
            if (need_mask) {
#pragma unroll
                for (int i = 0; i < TC_HALF; ++i)
                    if (key0 + i >= lim) v[i] = 0xff800000u;   // -inf
            }
            // P = 2^(S * scale - m) as packed bf16 (it will overwrite the first 32 columns of this half); returns the
            // sum of the half.  A row without a visible key so far has m = -inf: its P must be 0, not 2^(+inf).
            uint32_t pk[TC_HALF / 2];
            auto exps = [&](float m) {
                const float neg_m = (m == -INFINITY) ? 0.f : -m;
                const float2 sl2v = make_float2(sl2, sl2), nm = make_float2(neg_m, neg_m);
                float2 sum4[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
                for (int i = 0; i < TC_HALF / 2; ++i) {
                    const float2 x = ffma2(make_float2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1])), sl2v, nm);
                    float2 e;
                    e.x = fast_exp2(x.x);
                    e.y = fast_exp2(x.y);
                    sum4[i & 3] = fadd2(sum4[i & 3], e);
                    pk[i] = pack_bf16(e.x, e.y);
                }
                const float2 a = fadd2(sum4[0], sum4[1]), c = fadd2(sum4[2], sum4[3]);
                return (a.x + a.y) + (c.x + c.y);
            };
            // The exponentials are taken against the running maximum as it stands, without looking for the half's
            // own maximum first: (O, m, l) stay consistent whatever m is, and fp32 and bf16 carry the range.  Only when
            // the half's sum shows that some score lies far above m (or no key has been seen yet) is the maximum
            // raised, O rescaled and the half redone.  The decision is taken per warp: tensor-memory accesses are
            // warp-wide.
            float part_sum = 0.f;
            bool redo = m_run == -INFINITY;
            if (!__any_sync(0xffffffffu, redo)) {
                part_sum = exps(m_run);
                redo = !(part_sum < kSumLimit);              // also true for inf and NaN
            }
            if (__any_sync(0xffffffffu, redo)) {
                float mxc[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) mxc[c] = fmaxf(__uint_as_float(v[2 * c]), __uint_as_float(v[2 * c + 1]));
#pragma unroll
                for (int i = 16; i < TC_HALF; i += 16)
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        mxc[c] = fmax3(mxc[c], __uint_as_float(v[i + 2 * c]), __uint_as_float(v[i + 2 * c + 1]));
                const float mx = fmaxf(fmax3(mxc[0], mxc[1], mxc[2]), fmax3(fmax3(mxc[3], mxc[4], mxc[5]), mxc[6], mxc[7]));
                const float m_new = fmaxf(m_run, mx * sl2);
                // 0 on a row's first visible half; a row that has seen no key yet keeps (m, l) = (-inf, 0)
                const float alpha = (m_new == -INFINITY) ? 1.f : fast_exp2(m_run - m_new);
                l_run *= alpha;
                m_run = m_new;
                if (j > 0) {
                    // O must be quiescent: wait for the P V product of the previous half
                    mbar_wait(bar(BAR_PV_DONE + qt), (j - 1) & 1, wc);
                    tc_fence_after_sync();
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
                part_sum = exps(m_run);
            }
            tmem_st32(tS + u * 64, pk);
            l_run += part_sum;
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(BAR_P_READY + qt * 2 + u));
        }
        }

        // ---- epilogue: O / l  (or the unnormalised partial for the split merge)
        // (BAR_O_READY completes exactly once.)
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
                uint32_t o[32];
                tmem_ld32(tO + c0, o);
                tmem_wait_ld();
                if (row_ok) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint4 w;
                        w.x = pack_bf16(__uint_as_float(o[q4 * 8 + 0]) * inv, __uint_as_float(o[q4 * 8 + 1]) * inv);
                        w.y = pack_bf16(__uint_as_float(o[q4 * 8 + 2]) * inv, __uint_as_float(o[q4 * 8 + 3]) * inv);
                        w.z = pack_bf16(__uint_as_float(o[q4 * 8 + 4]) * inv, __uint_as_float(o[q4 * 8 + 5]) * inv);
                        w.w = pack_bf16(__uint_as_float(o[q4 * 8 + 6]) * inv, __uint_as_float(o[q4 * 8 + 7]) * inv);
                        *reinterpret_cast<uint4*>(dst + c0 + q4 * 8) = w;
                    }
                }
            }
        } else if (PAIR) {
            // ---- key list split in two, the two CTAs in one cluster (see the comment above the kernel).
            // CTA r finishes column half r of all 256 rows: it sends the other half of its partial and receives
            // the partner's half r.
            constexpr int DH = D / 2;
            constexpr int NCELL = DH / 4;              // 16-byte cells per half row
            constexpr uint32_t HALF_BYTES = TC_ROWS * DH * 4, ML_BYTES = TC_ROWS * 8;
            const int rl = qt * 128 + lane_base + lane;                       // row within the CTA
            // K/V stages: [0, HALF_BYTES) the half this CTA sends,
            // [HALF_BYTES, 2 HALF_BYTES) the half it receives; rows of DH fp32, cells XOR-swizzled by the row
            uint8_t* park = sK;
            static_assert(2 * STAGES * KV_TILE_BYTES >= 2 * HALF_BYTES, "both halves must fit");
            // both warpgroups have passed their O_READY: no MMA reads the Q tiles or the K/V stages any more
            asm volatile("bar.sync 1, 256;\n" ::: "memory");
            // shared memory of the Q tiles: warp w of Q tile q stages its bf16 result in the first half of the 8 KB
            // at q * 32 KB + w * 8 KB (D = 128); the unused half of the first slot holds this CTA's (m, l), that of the
            // second slot the partner's
            uint8_t* wslot = sQ + qt * Q_TILE_BYTES + (warp_u & 3) * (Q_TILE_BYTES / 4);
            float2* ml_mine = reinterpret_cast<float2*>(sQ + Q_TILE_BYTES / 8);                         // [256]
            float2* ml_other = reinterpret_cast<float2*>(sQ + Q_TILE_BYTES / 4 + Q_TILE_BYTES / 8);     // [256]
            static_assert(TC_ROWS * 8 <= 128 * D * 2 / 8, "(m, l) of 256 rows must fit in half a warp slot");
            const int h_mine = split, h_send = split ^ 1;
            if (tid == 0) mbar_arrive_expect_tx(bar(BAR_PAIR), HALF_BYTES + ML_BYTES);
            {
                float4* prow = reinterpret_cast<float4*>(park) + (size_t)rl * NCELL;
                if (n_tiles > 0) {
#pragma unroll
                    for (int c0 = 0; c0 < DH; c0 += 32) {
                        uint32_t o[32];
                        tmem_ld32(tO + h_send * DH + c0, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int q4 = 0; q4 < 8; ++q4)
                            prow[(c0 / 4 + q4) ^ (rl & (NCELL - 1))] =
                                make_float4(__uint_as_float(o[4 * q4]), __uint_as_float(o[4 * q4 + 1]),
                                            __uint_as_float(o[4 * q4 + 2]), __uint_as_float(o[4 * q4 + 3]));
                    }
                }
                ml_mine[rl] = make_float2(m_run, l_run);     // m = -inf: empty part
                fence_async_smem();                          // the bulk copies read these writes through the async proxy
            }
            cluster_arrive();
            cluster_wait();
            if (tid == 0) {
                const uint32_t other = split ^ 1;
                const uint32_t rbar = cluster_map(bar(BAR_PAIR), other);
                bulk_copy_to_cluster(cluster_map(smem_u32(ml_other), other), smem_u32(ml_mine), ML_BYTES, rbar);
                constexpr uint32_t PIECE = HALF_BYTES / 4;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    bulk_copy_to_cluster(cluster_map(smem_u32(park) + HALF_BYTES + i * PIECE, other), smem_u32(park) + i * PIECE, PIECE, rbar);
            }
            mbar_wait(bar(BAR_PAIR), 0, wc);
            cluster_arrive();                                // the partner's copies have landed here: it may go once it has them too
            {
                float4* stage = reinterpret_cast<float4*>(wslot);
                const int wrow0 = row0 + qt * 128 + lane_base;
                const int64_t own_off = (((int64_t)b * p.l_C + cq) * p.H + kvh * G + g) * D;
                const uint32_t own_lo = (uint32_t)own_off, own_hi = (uint32_t)(own_off >> 32);
                const float4* prow = reinterpret_cast<const float4*>(park + HALF_BYTES) + (size_t)rl * NCELL;
                const float2 mlo = ml_other[rl];
                // weights of the two parts in the log2 domain (Algorithm 1's merge of (O, m, l)); part 0 first in every sum
                const float m0 = split == 0 ? m_run : mlo.x, l0 = split == 0 ? l_run : mlo.y;
                const float m1 = split == 0 ? mlo.x : m_run, l1 = split == 0 ? mlo.y : l_run;
                const float m_max = fmaxf(m0, m1);
                const float w0 = (m0 == -INFINITY) ? 0.f : fast_exp2(m0 - m_max);
                const float w1 = (m1 == -INFINITY) ? 0.f : fast_exp2(m1 - m_max);
                const float inv = 1.f / (w0 * l0 + w1 * l1);
                const float a0 = w0 * inv, a1 = w1 * inv;
                const float a_own = split == 0 ? a0 : a1, a_oth = split == 0 ? a1 : a0;
                float acc[DH];
                if (split == 0) {
                    // acc = a0 * own, then += a1 * other
#pragma unroll
                    for (int cc = 0; cc < DH; cc += 16) {
                        uint32_t o[16];
                        tmem_ld16(tO + h_mine * DH + cc, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) acc[cc + i] = (a_own != 0.f) ? a_own * __uint_as_float(o[i]) : 0.f;
                    }
                    if (a_oth != 0.f) {                      // an empty part may hold anything
#pragma unroll
                        for (int c = 0; c < NCELL; ++c) {
                            const float4 val = prow[c ^ (rl & (NCELL - 1))];
                            acc[4 * c] = fmaf(a_oth, val.x, acc[4 * c]);
                            acc[4 * c + 1] = fmaf(a_oth, val.y, acc[4 * c + 1]);
                            acc[4 * c + 2] = fmaf(a_oth, val.z, acc[4 * c + 2]);
                            acc[4 * c + 3] = fmaf(a_oth, val.w, acc[4 * c + 3]);
                        }
                    }
                } else {
                    // the same sums in the same order: acc = a0 * other, then += a1 * own
#pragma unroll
                    for (int c = 0; c < NCELL; ++c) {
                        const float4 val = prow[c ^ (rl & (NCELL - 1))];
                        acc[4 * c] = (a_oth != 0.f) ? a_oth * val.x : 0.f;
                        acc[4 * c + 1] = (a_oth != 0.f) ? a_oth * val.y : 0.f;
                        acc[4 * c + 2] = (a_oth != 0.f) ? a_oth * val.z : 0.f;
                        acc[4 * c + 3] = (a_oth != 0.f) ? a_oth * val.w : 0.f;
                    }
#pragma unroll
                    for (int cc = 0; cc < DH; cc += 16) {
                        uint32_t o[16];
                        tmem_ld16(tO + h_mine * DH + cc, o);
                        tmem_wait_ld();
                        if (a_own != 0.f) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) acc[cc + i] = fmaf(a_own, __uint_as_float(o[i]), acc[cc + i]);
                        }
                    }
                }
                store_half_rows<DH>(acc, stage, lane, wrow0, R, own_lo, own_hi, p.O + h_mine * DH);
            }
            cluster_wait();
        } else {
            // ---- split key list.  Every CTA leaves its partial (O, m, l) in the scratch; the CTA that
            // finishes a (sequence, head, row tile) unit last combines the others' partials with its own,
            // which is still in tensor memory, and writes the rows of O: no CTA waits for another one.
            // Scratch of part s: O rows [Rp][D] fp32, then (m, l) pairs [Rp][2].
            constexpr int DH = D / 2;                  // columns handled per round
            constexpr int NC = DH / 4;                 // float4 per staged row: 16 or 8
            const int Rp = p.Rp;
            float* unit_base = p.part + (((int64_t)b * p.HG + kvh) * p.nsplit) * (int64_t)Rp * (D + 2);
            const int64_t part_stride = (int64_t)Rp * (D + 2);
            float* myO = unit_base + split * part_stride;
            // Staging for coalesced traffic: this warp's quarter of its own Q tile, 32 rows x DH fp32.
            // Free by now: O_READY covers every Q K^T of the tile.  16-byte cells are XOR-swizzled by
            // the row so that row-per-lane and row-per-half-warp accesses are both conflict-free.
            float4* stage = reinterpret_cast<float4*>(sQ + qt * Q_TILE_BYTES + (warp_u & 3) * (Q_TILE_BYTES / 4));
            const int wrow0 = row0 + qt * 128 + lane_base;        // first row of this warp
            int* cnt = p.unit_count + ((int64_t)b * p.HG + kvh) * gridDim.x + blockIdx.x;
            // When every other CTA of the unit has arrived already, this one merges straight from its
            // tensor memory and publishes nothing.
            asm volatile("bar.sync 1, 256;\n" ::: "memory");
            if (tid == 0) {
                const bool all_in = atomicAdd(cnt, 0) == p.nsplit - 1;
                if (all_in) *cnt = 0;                              // ready for the next launch
                merge_ticket = all_in ? p.nsplit - 1 : -1;
            }
            asm volatile("bar.sync 1, 256;\n" ::: "memory");
            if (merge_ticket != p.nsplit - 1) {
                if (n_tiles > 0) {
#pragma unroll 1
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int cc = 0; cc < DH; cc += 32) {
                            uint32_t o[32];
                            tmem_ld32(tO + h * DH + cc, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int q4 = 0; q4 < 8; ++q4)
                                stage[lane * NC + ((cc / 4 + q4) ^ (lane & (NC - 1)))] =
                                    make_float4(__uint_as_float(o[4 * q4]), __uint_as_float(o[4 * q4 + 1]),
                                                __uint_as_float(o[4 * q4 + 2]), __uint_as_float(o[4 * q4 + 3]));
                        }
                        __syncwarp();
#pragma unroll 4
                        for (int it = 0; it < NC; ++it) {
                            const int e = it * 32 + lane, rr = e / NC, c = e % NC;
                            const float4 val = stage[rr * NC + (c ^ (rr & (NC - 1)))];
                            if (wrow0 + rr < R)
                                __stcg(reinterpret_cast<float4*>(myO + (int64_t)(wrow0 + rr) * D + h * DH) + c, val);
                        }
                        __syncwarp();
                    }
                }
                if (row_ok) __stcg(reinterpret_cast<float2*>(myO + (int64_t)Rp * D) + row, make_float2(m_run, l_run));   // m = -inf: empty part
                __threadfence();
                asm volatile("bar.sync 1, 256;\n" ::: "memory");
                if (tid == 0) {
                    const int ticket = atomicAdd(cnt, 1);
                    if (ticket == p.nsplit - 1) *cnt = 0;
                    merge_ticket = ticket;
                }
                asm volatile("bar.sync 1, 256;\n" ::: "memory");
            }
            if (merge_ticket == p.nsplit - 1) {
                __threadfence();
                // The other parts' rows arrive through a ring of two shared-memory buffers per warp
                // (16-byte cp.async, all copies of a buffer in flight together), in the order
                // (column half, part).  The K/V stages serve as the ring: both warpgroups have passed
                // their O_READY before the arrival barrier above, so no MMA reads them any more.
                const int64_t own_off = (((int64_t)b * p.l_C + cq) * p.H + kvh * G + g) * D;     // this lane's row of O, in elements
                const uint32_t own_lo = (uint32_t)own_off, own_hi = (uint32_t)(own_off >> 32);
                constexpr int RING_BYTES = 2 * STAGES * KV_TILE_BYTES;
                static_assert(RING_BYTES / 8 >= 2 * 32 * (D / 8) * 16, "two buffers of 32 rows x D/2 floats per warp");
                float4* ring = reinterpret_cast<float4*>(sK + warp_u * (RING_BYTES / 8));
                const int n_other = p.nsplit - 1, n_pairs = 2 * n_other;
                auto other = [&](int i) { const int s = i % n_other; return s + (s >= split ? 1 : 0); };
                auto issue = [&](int i) {
                    const int h = i / n_other;
                    const float* srcO = unit_base + other(i) * part_stride + h * DH;
                    float4* buf = ring + (i & 1) * (32 * NC);
#pragma unroll
                    for (int it = 0; it < NC; ++it) {
                        const int e = it * 32 + lane, rr = e / NC, c = e % NC;
                        const bool ok = wrow0 + rr < R;
                        cp_async16(buf + rr * NC + (c ^ (rr & (NC - 1))), srcO + (int64_t)(ok ? wrow0 + rr : 0) * D + c * 4,
                                   ok ? 16 : 0);
                    }
                    cp_async_commit();
                };
                issue(0);
                if (n_pairs > 1) issue(1);
                // weights of the parts in the log2 domain (Algorithm 1's merge of (O, m, l))
                float w[kAttPrefillSplits];
                float m_max = m_run;
                float2 ml[kAttPrefillSplits];
#pragma unroll
                for (int s = 0; s < kAttPrefillSplits; ++s) {
                    ml[s] = make_float2(-INFINITY, 0.f);
                    if (s < p.nsplit && s != split && row_ok)
                        ml[s] = __ldcg(reinterpret_cast<const float2*>(unit_base + s * part_stride + (int64_t)Rp * D) + row);
                    if (s == split) ml[s] = make_float2(m_run, l_run);
                    m_max = fmaxf(m_max, ml[s].x);
                }
                float den = 0.f;
#pragma unroll
                for (int s = 0; s < kAttPrefillSplits; ++s) {
                    w[s] = (ml[s].x == -INFINITY) ? 0.f : fast_exp2(ml[s].x - m_max);
                    den += w[s] * ml[s].y;
                }
                const float inv = 1.f / den;
                auto pick = [&](int s) { return s == 0 ? w[0] : s == 1 ? w[1] : s == 2 ? w[2] : w[3]; };   // no dynamic register indexing
#pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    // The parts are added in split order whichever CTA happens to merge (its own part comes
                    // from tensor memory, the others from the ring), so the result does not depend on the
                    // order of arrival: the same bits as a merge pass over all parts.
                    float acc[DH];
#pragma unroll
                    for (int i = 0; i < DH; ++i) acc[i] = 0.f;
                    auto add_own = [&]() {
                        const float wo = pick(split) * inv;       // 0 when this CTA's own part is empty
#pragma unroll
                        for (int cc = 0; cc < DH; cc += 16) {
                            uint32_t o[16];
                            tmem_ld16(tO + h * DH + cc, o);
                            tmem_wait_ld();
                            if (wo != 0.f) {
#pragma unroll
                                for (int i = 0; i < 16; ++i) acc[cc + i] = fmaf(wo, __uint_as_float(o[i]), acc[cc + i]);
                            }
                        }
                    };
                    int k = 0;                                    // index among the other parts
#pragma unroll 1
                    for (int sp = 0; sp < p.nsplit; ++sp) {
                        if (sp == split) {
                            add_own();
                            continue;
                        }
                        const int i = h * n_other + k;
                        ++k;
                        if (i + 1 < n_pairs) cp_async_wait<1>();
                        else cp_async_wait<0>();
                        __syncwarp();
                        const float4* buf = ring + (i & 1) * (32 * NC);
                        const float ws = pick(sp) * inv;
#pragma unroll
                        for (int c = 0; c < NC; ++c) {
                            const float4 val = buf[lane * NC + (c ^ (lane & (NC - 1)))];
                            if (ws != 0.f) {                     // an empty part may hold anything
                                acc[4 * c] = fmaf(ws, val.x, acc[4 * c]);
                                acc[4 * c + 1] = fmaf(ws, val.y, acc[4 * c + 1]);
                                acc[4 * c + 2] = fmaf(ws, val.z, acc[4 * c + 2]);
                                acc[4 * c + 3] = fmaf(ws, val.w, acc[4 * c + 3]);
                            }
                        }
                        __syncwarp();
                        if (i + 2 < n_pairs) issue(i + 2);
                    }
                    store_half_rows<D / 2>(acc, stage, lane, wrow0, R, own_lo, own_hi, p.O + h * DH);
                }
            }
        }
    } else if (warp_u < TC_MMA_WARP) {
        // ------------------------------------------------------------ producers: Q, then K/V tiles
        const int ptid = tid - TC_SOFTMAX_WARPS * 32;      // 0..127
        if (has_work && p.q_tma) {
            // two boxes per 64-column block: rows (query, head-in-group) of one key/value head
            if (ptid == 0) {
                mbar_arrive_expect_tx(bar(BAR_Q_FULL), 2 * Q_TILE_BYTES);
                const CUtensorMap* qm = far ? &qgmap : &qmap;
#pragma unroll
                for (int qt = 0; qt < 2; ++qt)
#pragma unroll
                    for (int blk = 0; blk < D / 64; ++blk)
                        tma_load_3d(smem_u32(sQ + qt * Q_TILE_BYTES + blk * Q_BLK_BYTES), qm, blk * 64, kvh * G,
                                    b * p.l_C + (row0 + qt * 128) / G, bar(BAR_Q_FULL));
            }
        } else if (has_work) {
            // group sizes that do not divide 128: 16-byte copies, row by row
            const int chunk = ptid % CH, rsub = ptid / CH, cin = chunk & 7;
            constexpr int RSTEP = TC_PRODUCERS / CH;
            const __nv_bfloat16* Qsrc = far ? p.Qg : p.Q;
            for (int r = rsub; r < TC_ROWS; r += RSTEP) {
                const int row = row0 + r;
                const bool ok = row < R;
                const int cq = ok ? row / G : 0, g = ok ? row % G : 0;
                const int64_t qoff = (((int64_t)b * p.l_C + cq) * p.H + kvh * G + g) * D + chunk * 8;
                const int rr = r & 127;
                const uint32_t doff = (r >> 7) * Q_TILE_BYTES + (chunk >> 3) * Q_BLK_BYTES + rr * 128 + ((cin ^ (rr & 7)) << 4);
                cp_async16(sQ + doff, Qsrc + qoff, ok ? 16 : 0);
            }
            cp_async_arrive_noinc(bar(BAR_Q_FULL));
        }
        // K/V tiles: four threads share a row (one instruction of the four covers 64 contiguous bytes of it: whole
        // sectors), so a thread works out the cache position of four rows per 128-key tile, not of sixteen, and
        // copies CH / 4 chunks of each; the loop is sensitive to the instructions the CTA's warps issue, these included.
        constexpr int TPR = 4;                             // threads per row
        constexpr int RPP = TC_PRODUCERS / TPR;            // rows per pass: 32
        constexpr int NPASS = TC_BN / RPP;                 // 4
        constexpr int CPT = CH / TPR;                      // chunks per thread and row: 4 (D = 128) or 2
        const int q4 = ptid % TPR, rfirst = ptid / TPR;
        const __nv_bfloat16* Kb0 = p.K + ((int64_t)b * p.max_tokens * p.HG + kvh) * D + q4 * 8;
        const __nv_bfloat16* Kb1 = p.Kg + ((int64_t)b * p.max_tokens * p.HG + kvh) * D + q4 * 8;
        const __nv_bfloat16* Vb = p.V + ((int64_t)b * p.max_tokens * p.HG + kvh) * D + q4 * 8;
        const int32_t* idx = p.idx + (int64_t)b * p.top_k;
        const int64_t tok_stride = (int64_t)p.HG * D;
        // chunk c = TPR i + q4 of row r goes to block (c >> 3), byte r * 128 + (((c & 7) ^ (r & 7)) << 4) of the tile
        uint32_t row_off[NPASS];
#pragma unroll
        for (int it = 0; it < NPASS; ++it) {
            const int r = rfirst + it * RPP;
            row_off[it] = (uint32_t)(r * 128) | (uint32_t)((r & 7) << 4);      // XOR with (c & 7) << 4 gives the swizzled chunk
        }
        int bad_idx = 0;
#pragma unroll 1
        for (int phase = 0; phase < 2; ++phase) {
        if (phase == 1 && !planned) plan();
        const KeyList kl = phase == 0 ? list_early : list_late;
        const int j_first = phase == 0 ? 0 : n_early, j_last = phase == 0 ? n_early : n_tiles;
        const int key_first = phase == 0 ? early_begin * TC_BN : part_lo + tile_begin * TC_BN;
        for (int j = j_first; j < j_last; ++j) {
            const int s = j % STAGES;
            const uint32_t ph = ((j / STAGES) & 1) ^ 1;
            const int key0 = key_first + (j - j_first) * TC_BN;
            int pos[NPASS];
            uint32_t from_idx = 0;                      // rows whose position was read from the selection
#pragma unroll
            for (int it = 0; it < NPASS; ++it) {
                const int jj = key0 + rfirst + it * RPP;
                int q = -1;
                if (jj >= kl.row_lim) q = -1;
                else if (p.staged || jj < kl.ie) q = jj;
                else if (jj < kl.ng) {
                    q = __ldg(idx + (jj - kl.ie));
                    from_idx |= 1u << it;
                } else q = kl.me + (jj - kl.ng);
                pos[it] = q;
            }
            mbar_wait(bar(BAR_K_EMPTY + s), ph, wc);
            // (the range check of the selected positions comes after the wait: the index loads above stay in
            // flight across it instead of being consumed at once)
#pragma unroll
            for (int it = 0; it < NPASS; ++it)
                if ((from_idx >> it) & 1u) pos[it] = clamp_selected(pos[it], i_end, m_end, bad_idx);
#pragma unroll
            for (int it = 0; it < NPASS; ++it) {
                const __nv_bfloat16* src = (far ? Kb1 : Kb0) + (pos[it] < 0 ? 0 : pos[it]) * tok_stride;
                const int nbytes = pos[it] < 0 ? 0 : 16;
                uint8_t* tile = sK + s * KV_TILE_BYTES;
#pragma unroll
                for (int i = 0; i < CPT; ++i) {
                    const int c = i * TPR;                  // + q4: the chunk; TPR divides 8, so (c + q4) >> 3 = c >> 3 and (c + q4) & 7 = (c & 7) + q4
                    cp_async16(tile + (c >> 3) * KV_BLK_BYTES + (row_off[it] ^ (uint32_t)(((c & 7) + q4) << 4)), src + c * 8, nbytes);
                }
            }
            cp_async_arrive_noinc(bar(BAR_K_FULL + s));
            mbar_wait(bar(BAR_V_EMPTY + s), ph, wc);
#pragma unroll
            for (int it = 0; it < NPASS; ++it) {
                const __nv_bfloat16* src = Vb + (pos[it] < 0 ? 0 : pos[it]) * tok_stride;
                const int nbytes = pos[it] < 0 ? 0 : 16;
                uint8_t* tile = sV + s * KV_TILE_BYTES;
#pragma unroll
                for (int i = 0; i < CPT; ++i) {
                    const int c = i * TPR;
                    cp_async16(tile + (c >> 3) * KV_BLK_BYTES + (row_off[it] ^ (uint32_t)(((c & 7) + q4) << 4)), src + c * 8, nbytes);
                }
            }
            cp_async_arrive_noinc(bar(BAR_V_FULL + s));
        }
        }
        if (bad_idx) atomicExch(p.status, kStatusBadIndex);
        cp_async_wait<0>();
    } else if (warp_u == TC_MMA_WARP && has_work) {
        // ------------------------------------------------------------ MMA issue: one converged warp, lane 0 leads.
        // The fixed order (Q tile 0's products of a tile, then Q tile 1's) keeps the two Q tiles half a period
        // apart: S of Q tile 1 always becomes ready one block of products after S of Q tile 0, so each softmax
        // warpgroup computes while the tensor core works for the other one.  (Two independent issuing warps settle
        // into lockstep instead: both softmaxes, then both blocks.)
        const uint32_t lead = lane == 0;
        constexpr uint32_t ID_QK = idesc_bf16(128, TC_BN, false, false);
        constexpr uint32_t ID_PV = idesc_bf16(128, D, false, true);
        const uint32_t hi = desc_hi_sw128();
        const uint32_t qlo = desc_lo_kmajor(smem_u32(sQ));
        const uint32_t klo = desc_lo_kmajor(smem_u32(sK)), vlo = desc_lo_mnmajor(smem_u32(sV), KV_BLK_BYTES);
        // descriptor low words advance by compile-time constants (bytes >> 4)
        auto issue_qk = [&](int qt, int s) {                // S[qt] = Q[qt] . K[s]^T, 128 keys
            const uint32_t a0 = qlo + qt * (Q_TILE_BYTES >> 4);
            const uint32_t b0 = klo + s * (KV_TILE_BYTES >> 4);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks)
                umma_ss(tmem + qt * 128, a0 + (((ks >> 2) * Q_BLK_BYTES + (ks & 3) * 32) >> 4),
                        b0 + (((ks >> 2) * KV_BLK_BYTES + (ks & 3) * 32) >> 4), hi, ID_QK, ks, lead);
        };
        auto issue_pv = [&](int qt, int s, int u, int acc) { // O[qt] (+)= P[qt][half u] . V[s][keys of half u]
            const uint32_t b0 = vlo + s * (KV_TILE_BYTES >> 4) + u * ((TC_HALF * 128) >> 4);
#pragma unroll
            for (int ks = 0; ks < TC_HALF / 16; ++ks)
                umma_ts(tmem + 256 + qt * D, tmem + qt * 128 + u * 64 + ks * 8, b0 + ks * (2048 >> 4), hi, ID_PV, acc | ks, lead);
        };
        mbar_wait(bar(BAR_Q_FULL), 0, wc);
        mbar_wait(bar(BAR_K_FULL + 0), 0, wc);
        fence_async_smem();
        tc_fence_after_sync();
        issue_qk(0, 0);
        umma_commit(bar(BAR_S_READY + 0), lead);
        issue_qk(1, 0);
        umma_commit(bar(BAR_S_READY + 1), lead);
        umma_commit(bar(BAR_K_EMPTY + 0), lead);
        for (int T = 0; !planned || T < n_tiles; ++T) {
            const int s = T % STAGES;
            const int Tn = T + 1, sn = Tn % STAGES;
            // Whether a tile follows the last early one is known only after the wait for the preceding kernel: this
            // warp takes the wait at the start of that tile's round (by then the preceding kernel has finished, unless
            // the early list is short), so that the round can issue the first late tile's products like any other.
            if (!planned && Tn >= n_early) plan();
            const bool more = !planned || Tn < n_tiles;
            mbar_wait(bar(BAR_V_FULL + s), (T / STAGES) & 1, wc);
            fence_async_smem();
#pragma unroll
            for (int qt = 0; qt < 2; ++qt) {
                mbar_wait(bar(BAR_P_READY + qt * 2 + 0), T & 1, wc);
                tc_fence_after_sync();
                issue_pv(qt, s, 0, T > 0);
                umma_commit(bar(BAR_PV_DONE + qt), lead);
                if (more && qt == 0) {
                    mbar_wait(bar(BAR_K_FULL + sn), (Tn / STAGES) & 1, wc);
                    fence_async_smem();
                }
                mbar_wait(bar(BAR_P_READY + qt * 2 + 1), T & 1, wc);
                tc_fence_after_sync();
                issue_pv(qt, s, 1, 1);
                umma_commit(bar(BAR_PV_DONE + qt), lead);
                if (!more) umma_commit(bar(BAR_O_READY + qt), lead);
                if (qt == 1) umma_commit(bar(BAR_V_EMPTY + s), lead);
                if (more) {
                    issue_qk(qt, sn);         // overwrites S and P of this tile after the P V products above, in issue order
                    umma_commit(bar(BAR_S_READY + qt), lead);
                    if (qt == 1) umma_commit(bar(BAR_K_EMPTY + sn), lead);
                }
            }
        }
    }

    if (PAIR && warp_u >= TC_SOFTMAX_WARPS) {
        // the cluster barriers count every thread: the warps with nothing to publish pass both
        cluster_arrive();
        cluster_wait();
        cluster_arrive();
        cluster_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

}  // namespace

template <int D, bool PAIR>
static cudaError_t launch_tc_kernel(esa_ctx* ctx, const CUtensorMap& qmap, const CUtensorMap& qgmap, const TcAttendParams& p,
                                    dim3 grid, cudaStream_t st, bool probe_only) {
    constexpr int smem = 2 * 128 * D * 2 + 2 * TC_STAGES * TC_BN * D * 2 + 1024;
    cudaError_t e = cudaFuncSetAttribute(attend_tc_kernel<D, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    // the in-kernel register split assumes the launch allocation it was sized for
    static int regs_checked = 0;
    if (!regs_checked) {
        cudaFuncAttributes fa;
        e = cudaFuncGetAttributes(&fa, attend_tc_kernel<D, PAIR>);
        if (e != cudaSuccess) return e;
        if (fa.numRegs != TC_REGS_LAUNCH) return cudaErrorInvalidConfiguration;
        regs_checked = 1;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 2;
    cfg.attrs = attr;
    cfg.numAttrs = PAIR ? 2 : 1;
    if (probe_only) {
        // can the device place a pair of these CTAs at all?
        int n_clusters = 0;
        e = cudaOccupancyMaxActiveClusters(&n_clusters, attend_tc_kernel<D, PAIR>, &cfg);
        if (e != cudaSuccess) return e;
        return n_clusters > 0 ? cudaSuccess : cudaErrorNotSupported;
    }
    return cudaLaunchKernelEx(&cfg, attend_tc_kernel<D, PAIR>, qmap, qgmap, p);
}

template <int D>
static cudaError_t launch_tc(esa_ctx* ctx, TcAttendParams& p, int B, int n_att_max, cudaStream_t st, int* nsplit_out) {
    const int R = p.l_C * p.G;
    const int row_tiles = (R + TC_ROWS - 1) / TC_ROWS;
    p.Rp = (R + 1) & ~1;
    if ((size_t)B * p.HG * row_tiles > ctx->att_count_elems) return cudaErrorNotSupported;
    // Split the key list when that fills the machine better: cost model = waves x tiles per CTA
    // (+ half a tile-equivalent of fixed work per CTA), one CTA per SM.  Two-position attention needs an even
    // number of splits (one group per part); its longer part sets the tiles per CTA.
    const int ctas = row_tiles * p.HG * B;
    const int n_tiles = (n_att_max + TC_BN - 1) / TC_BN;
    int i_end_max = 0;
    for (int b = 0; b < B; ++b) i_end_max = max(i_end_max, p.meta.i_end[b]);
    const int far_tiles = min(n_tiles, (i_end_max + p.top_k + TC_BN - 1) / TC_BN);
    const int step = p.two ? 2 : 1;
    int best = 0;
    double best_cost = 1e30;
    for (int ns = step; ns <= kAttPrefillSplits && (ns <= n_tiles || best == 0); ns += step) {
        if ((size_t)B * p.HG * ns * p.Rp * (D + 2) > ctx->att_part_elems) break;
        const int grp = p.two ? ns / 2 : ns;
        const int longest = p.two ? max(far_tiles, n_tiles - far_tiles + 1) : n_tiles;
        const int per = (longest + grp - 1) / grp;
        const int waves = (ctas * ns + ctx->num_sms - 1) / ctx->num_sms;
        const double cost = (double)waves * (per + 0.5) + (ns > 1 ? 0.25 * ns : 0.0);
        if (cost < best_cost - 1e-9) { best_cost = cost; best = ns; }
    }
    if (best == 0) return cudaErrorNotSupported;
    p.nsplit = best;
    *nsplit_out = best;
    CUtensorMap qmap, qgmap;
    p.q_tma = make_tensor_map_q(&qmap, p.Q, (uint64_t)B * p.l_C, p.H, D, p.G) ? 1 : 0;
    if (p.q_tma && p.two) p.q_tma = make_tensor_map_q(&qgmap, p.Qg, (uint64_t)B * p.l_C, p.H, D, p.G) ? 1 : 0;
    if (!p.q_tma) memset(&qmap, 0, sizeof(qmap));
    if (!p.q_tma || !p.two) memset(&qgmap, 0, sizeof(qgmap));
    const dim3 grid(row_tiles, p.HG, B * best);
    // a two-way split runs as CTA pairs that merge through distributed shared memory, where the device can place pairs
    static int pair_ok = -1;                                 // per instantiation; probed once
    if (best == 2 && pair_ok < 0) pair_ok = launch_tc_kernel<D, true>(ctx, qmap, qgmap, p, grid, st, true) == cudaSuccess ? 1 : 0;
    ProfScope prof(ctx, KC_ATTEND_TC, st);
    cudaError_t e = (best == 2 && pair_ok == 1) ? launch_tc_kernel<D, true>(ctx, qmap, qgmap, p, grid, st, false)
                                                : launch_tc_kernel<D, false>(ctx, qmap, qgmap, p, grid, st, false);
    ctx->launches += 1;
    return e;
}

// Returns cudaErrorNotSupported when this path does not cover the shape (the caller then
// uses the split kernel); nsplit_out reports how many ways the key list was split (merged in-kernel).
cudaError_t launch_attend_tc(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* Q, const __nv_bfloat16* Qg,
                             const __nv_bfloat16* K, const __nv_bfloat16* Kg, const __nv_bfloat16* V, const SeqMeta& meta,
                             const int32_t* idx, const int32_t* n_sel, __nv_bfloat16* O, int n_att_max, cudaStream_t st,
                             int* nsplit_out, int64_t cache_rows, bool staged) {
    const bool two = Qg != nullptr || Kg != nullptr;
    TcAttendParams p;
    p.Q = Q; p.K = K; p.Qg = Qg ? Qg : Q; p.Kg = Kg ? Kg : K;
    p.V = V; p.O = O; p.idx = idx; p.n_sel = n_sel; p.part = ctx->att_part; p.status = ctx->status;
    p.unit_count = ctx->att_count;
    p.staged = staged ? 1 : 0;
    p.two = two ? 1 : 0;
    p.early = ctx->attend_early && !two && !staged ? 1 : 0;
    p.max_tokens = cache_rows > 0 ? cache_rows : ctx->cfg.max_tokens; p.l_C = l_C; p.H = ctx->H; p.HG = ctx->HG; p.G = ctx->G;
    p.top_k = ctx->cfg.top_k; p.nsplit = 1;
    p.scale_log2 = ctx->scale * 1.4426950408889634f;
    p.meta = meta;
    if (ctx->d == 128) return launch_tc<128>(ctx, p, B, n_att_max, st, nsplit_out);
    if (ctx->d == 64) return launch_tc<64>(ctx, p, B, n_att_max, st, nsplit_out);
    return cudaErrorNotSupported;
}

}  // namespace esa
