// Eq. 5 on the 5th-generation tensor cores: Y = bf16(X W^T + b) for the two linear compressors.
//
// X is [rows, d_in] and W is [d', d_in], both with the reduction dimension contiguous, so both
// are K-major operands fetched by TMA in 128-column chunks (64-column boxes, 128-byte swizzle).
// The output is only d' wide, so a chunk of a few hundred rows gives a handful of 128-row
// tiles: the reduction dimension is split across the CTAs of a thread-block cluster (up to 16),
// every CTA puts all of its operand chunks in flight at once, accumulates its slice in tensor
// memory, parks the fp32 partial tile in its shared memory, and the cluster adds the partials
// through distributed shared memory in split order (deterministic), adds the bias, rounds to
// bf16 and scatters the rows to their cache positions.  No global scratch.
//
// Warp roles: warp 0 issues the TMA loads, warp 1 the MMAs (converged, lane 0 leads), warps
// 2-5 move the accumulator from tensor memory to shared memory; all six reduce.
#include <cooperative_groups.h>

#include "esa_internal.h"
#include "esa_umma.cuh"

namespace cg = cooperative_groups;

namespace esa {

namespace {

constexpr int CT_ROWS = 128;       // rows per CTA
constexpr int CT_KCHUNK = 128;     // reduction columns per pipeline stage
constexpr int CT_STAGES = 3;
constexpr int CT_THREADS = 192;
constexpr int CT_MAX_SPLIT = 16;

enum { CB_FULL = 0, CB_EMPTY = CB_FULL + CT_STAGES, CB_ACC = CB_EMPTY + CT_STAGES, CB_COUNT = CB_ACC + 1 };

struct CompressTcParams {
    const float* bias;
    __nv_bfloat16* dst;
    int* status;
    int rows, rows_per_seq, kslice;
    uint32_t* zero_words;      // optional: words the first CTA clears (the caller's next kernel accumulates there)
    int zero_count;
    int64_t seq_stride;
    RowMap map;
};

template <int DC>
__global__ void __launch_bounds__(CT_THREADS, 1)
compress_tc_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap,
                   CompressTcParams p) {
    constexpr int X_BYTES = CT_ROWS * CT_KCHUNK * 2;      // one stage of X: 2 blocks of [128][128 B]
    constexpr int W_BYTES = DC * CT_KCHUNK * 2;           // one stage of W: 2 blocks of [DC][128 B]
    constexpr int STAGE_BYTES = X_BYTES + W_BYTES;
    constexpr int PSTRIDE = DC + 4;                       // fp32 partial row stride (16-byte stores without bank conflicts)

    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    float* sPart = reinterpret_cast<float*>(smem);        // reuses the operand stages once the MMAs are done
    __shared__ uint64_t bars[CB_COUNT];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int row0 = blockIdx.x * CT_ROWS;
    const int split = blockIdx.y, nsplit = gridDim.y;
    const int k_begin = split * p.kslice;
    const int n_chunks = p.kslice / CT_KCHUNK;

    WaitCtx wc{&abort_flag, p.status};
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < CT_STAGES; ++s) {
            mbar_init(bar(CB_FULL + s), 1);
            mbar_init(bar(CB_EMPTY + s), 1);
        }
        mbar_init(bar(CB_ACC), 1);
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), DC < 32 ? 32 : DC);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    pdl_wait();
    pdl_launch_dependents();

    if (p.zero_words && blockIdx.x == 0 && blockIdx.y == 0)
        for (int i = tid; i < p.zero_count; i += CT_THREADS) p.zero_words[i] = 0u;
    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&xmap);
            tma_prefetch_desc(&wmap);
            for (int i = 0; i < n_chunks; ++i) {
                const int s = i % CT_STAGES;
                mbar_wait(bar(CB_EMPTY + s), ((i / CT_STAGES) & 1) ^ 1, wc);
                mbar_arrive_expect_tx(bar(CB_FULL + s), STAGE_BYTES);
                uint8_t* sx = smem + s * STAGE_BYTES;
                uint8_t* sw = sx + X_BYTES;
                const int k0 = k_begin + i * CT_KCHUNK;
#pragma unroll
                for (int blk = 0; blk < 2; ++blk) {
                    tma_load_2d(smem_u32(sx + blk * (CT_ROWS * 128)), &xmap, k0 + blk * 64, row0, bar(CB_FULL + s));
                    tma_load_2d(smem_u32(sw + blk * (DC * 128)), &wmap, k0 + blk * 64, 0, bar(CB_FULL + s));
                }
            }
        }
    } else if (warp == 1) {
        const uint32_t lead = lane == 0;
        const uint32_t hi = desc_hi_sw128();
        constexpr uint32_t IDESC = idesc_bf16(128, DC, false, false);
        for (int i = 0; i < n_chunks; ++i) {
            const int s = i % CT_STAGES;
            mbar_wait(bar(CB_FULL + s), (i / CT_STAGES) & 1, wc);
            tc_fence_after_sync();
            const uint32_t xlo = desc_lo_kmajor(smem_u32(smem + s * STAGE_BYTES));
            const uint32_t wlo = desc_lo_kmajor(smem_u32(smem + s * STAGE_BYTES + X_BYTES));
#pragma unroll
            for (int ks = 0; ks < CT_KCHUNK / 16; ++ks)
                umma_ss(tmem, xlo + (((ks >> 2) * (CT_ROWS * 128) + (ks & 3) * 32) >> 4),
                        wlo + (((ks >> 2) * (DC * 128) + (ks & 3) * 32) >> 4), hi, IDESC, (i > 0) | ks, lead);
            umma_commit(bar(CB_EMPTY + s), lead);
        }
        umma_commit(bar(CB_ACC), lead);
    } else {
        // accumulator -> this CTA's shared memory (after every MMA, hence every operand read, is done)
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;
        mbar_wait(bar(CB_ACC), 0, wc);
        tc_fence_after_sync();
#pragma unroll
        for (int c0 = 0; c0 < DC; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(tmem_addr(tmem, quarter * 32, c0), v);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<uint4*>(sPart + r * PSTRIDE + c0 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
    }

    // Every CTA of the cluster now holds the partial of its reduction slice.  Each sums a band of
    // rows over all of them in split order, adds the bias and rounds.
    cg::cluster_group cluster = cg::this_cluster();
    tc_fence_before_sync();
    cluster.sync();
    const int band = CT_ROWS / nsplit;
    constexpr int PER_ROW = DC / 4;
    for (int i = tid; i < band * PER_ROW; i += CT_THREADS) {
        const int lr = split * band + i / PER_ROW, c4 = (i % PER_ROW) * 4;
        const int row = row0 + lr;
        if (row >= p.rows) continue;
        // all remote reads of an element in flight together (a read from another CTA's shared memory takes most of
        // a microsecond); the sum order stays split order
        float4 v[CT_MAX_SPLIT];
#pragma unroll
        for (int j = 0; j < CT_MAX_SPLIT; ++j)
            v[j] = j < nsplit ? *reinterpret_cast<const float4*>(cluster.map_shared_rank(sPart, j) + lr * PSTRIDE + c4)
                              : make_float4(0.f, 0.f, 0.f, 0.f);
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < CT_MAX_SPLIT; ++j) {
            s.x += v[j].x; s.y += v[j].y; s.z += v[j].z; s.w += v[j].w;
        }
        if (p.bias) {
            s.x += p.bias[c4]; s.y += p.bias[c4 + 1]; s.z += p.bias[c4 + 2]; s.w += p.bias[c4 + 3];
        }
        const int b = row / p.rows_per_seq, ii = row % p.rows_per_seq;
        __nv_bfloat16* o = p.dst + ((int64_t)b * p.seq_stride + p.map.row0[b] + ii) * DC + c4;
        *reinterpret_cast<uint2*>(o) = make_uint2(pack_bf16(s.x, s.y), pack_bf16(s.z, s.w));
    }
    cluster.sync();    // shared memory stays alive until every remote read is done
    if (warp == 1) tmem_dealloc(tmem, DC < 32 ? 32 : DC);
}

template <int DC>
cudaError_t launch_t(esa_ctx* ctx, const __nv_bfloat16* X, int rows, int rows_per_seq, int d_in, const CUtensorMap* wmap,
                     const float* bias, __nv_bfloat16* dst, int64_t seq_stride, const RowMap& map, uint32_t* zero_words,
                     int zero_count, cudaStream_t st, bool small_grid) {
    CUtensorMap xmap;
    if (!make_tensor_map_bf16(&xmap, X, (uint64_t)rows, (uint64_t)d_in, CT_ROWS)) return cudaErrorNotSupported;
    const int row_tiles = (rows + CT_ROWS - 1) / CT_ROWS;
    const int n_chunks_total = d_in / CT_KCHUNK;
    // split the reduction while that still adds CTAs usefully (power of two, at most 16, whole chunks).  A call
    // whose result is not needed at once stays within an eighth of the SMs: beside the kernels of a step on another
    // stream it then fits on the SMs those leave idle (the attention grid of the Llama-3-8B shape leaves 20 of 148)
    // instead of holding back CTAs of theirs: 32 -> 16 CTAs for a 512-row chunk, +3 % prefill rate.
    const int cta_limit = small_grid ? max(ctx->num_sms / 8, 1) : ctx->num_sms;
    int nsplit = 1;
    while (nsplit < CT_MAX_SPLIT && n_chunks_total % (nsplit * 2) == 0 &&
           (small_grid ? row_tiles * nsplit * 2 <= cta_limit : row_tiles * nsplit < cta_limit))
        nsplit *= 2;
    constexpr int smem_stage = (CT_ROWS + DC) * CT_KCHUNK * 2;
    constexpr int smem_part = CT_ROWS * (DC + 4) * 4;
    constexpr int smem = (CT_STAGES * smem_stage > smem_part ? CT_STAGES * smem_stage : smem_part) + 1024;
    cudaError_t e = cudaFuncSetAttribute(compress_tc_kernel<DC>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(compress_tc_kernel<DC>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    // a cluster of 16 is beyond the portable size: use it only where the device can place one
    static int max_split = 0;
    if (!max_split) {
        max_split = 8;
        cudaLaunchConfig_t probe = {};
        probe.gridDim = dim3(1, CT_MAX_SPLIT);
        probe.blockDim = dim3(CT_THREADS);
        probe.dynamicSmemBytes = smem;
        cudaLaunchAttribute pa[1];
        pa[0].id = cudaLaunchAttributeClusterDimension;
        pa[0].val.clusterDim.x = 1;
        pa[0].val.clusterDim.y = CT_MAX_SPLIT;
        pa[0].val.clusterDim.z = 1;
        probe.attrs = pa;
        probe.numAttrs = 1;
        int n_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&n_clusters, compress_tc_kernel<DC>, &probe) == cudaSuccess && n_clusters > 0)
            max_split = CT_MAX_SPLIT;
        else
            cudaGetLastError();
    }
    while (nsplit > max_split) nsplit /= 2;
    CompressTcParams p;
    p.bias = bias; p.dst = dst; p.status = ctx->status; p.rows = rows; p.rows_per_seq = rows_per_seq;
    p.kslice = d_in / nsplit; p.seq_stride = seq_stride; p.map = map;
    p.zero_words = zero_words; p.zero_count = zero_count;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(row_tiles, nsplit);
    cfg.blockDim = dim3(CT_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = nsplit;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    ProfScope prof(ctx, KC_COMPRESS_TC, st);
    e = cudaLaunchKernelEx(&cfg, compress_tc_kernel<DC>, xmap, *wmap, p);
    ctx->launches += 1;
    return e;
}

}  // namespace

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up at run time so that the library carries no link-time
// dependency on libcuda.
static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

bool make_tensor_map_bf16(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || cols % 64 || box_rows == 0 || box_rows > 256 || (reinterpret_cast<uintptr_t>(base) & 15)) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t es[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Q as a 3-D tensor [B * l_C, H, D] read in boxes of (128 / G queries) x (G heads) x 64 columns: the rows
// of a box land in shared memory in (query, head-in-group) order, 128 bytes each, 128-byte swizzled.
bool make_tensor_map_q(CUtensorMap* map, const void* base, uint64_t n_queries, int H, int D, int G) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || G <= 0 || 128 % G || D % 64 || (reinterpret_cast<uintptr_t>(base) & 15)) return false;
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)n_queries};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)H * D * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)(128 / G)};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_compress_tc(esa_ctx* ctx, const __nv_bfloat16* X, int B, int rows_per_seq, int d_in,
                               const CUtensorMap* wmap, const float* bias, __nv_bfloat16* dst,
                               int64_t dst_seq_stride, const RowMap& map, uint32_t* zero_words, int zero_count,
                               cudaStream_t st, bool small_grid) {
    if (d_in % CT_KCHUNK) return cudaErrorNotSupported;
    const int rows = B * rows_per_seq;
    if (ctx->dc == 128) return launch_t<128>(ctx, X, rows, rows_per_seq, d_in, wmap, bias, dst, dst_seq_stride, map, zero_words, zero_count, st, small_grid);
    if (ctx->dc == 64) return launch_t<64>(ctx, X, rows, rows_per_seq, d_in, wmap, bias, dst, dst_seq_stride, map, zero_words, zero_count, st, small_grid);
    return cudaErrorNotSupported;
}

}  // namespace esa
