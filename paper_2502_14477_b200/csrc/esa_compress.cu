// Eq. 5: the linear compressors q' = f_q(q), k' = f_k(k) as a split-K bf16 GEMM with fp32
// accumulation, plus the K/V cache append.
//
//   Y[r, j] = bf16( sum_i X[r, i] * W[j, i] + bias[j] )
//
// X is [rows, d_in] (heads concatenated, Section 3.1 "Efficient Selection"), W is
// [d_c, d_in]; both are K-major, so the product is a TN GEMM.  The output is only d_c
// wide, so a chunk yields very few output tiles; the reduction dimension is therefore
// split across the CTAs of a thread-block cluster; each keeps its fp32 partial tile in
// shared memory and the cluster adds the partials through distributed shared memory in a
// fixed order (deterministic), adds the bias and rounds to bf16.  No global scratch.
#include <cooperative_groups.h>

#include "esa_internal.h"

namespace cg = cooperative_groups;

namespace esa {

constexpr int CP_BM = 64;   // rows per CTA (4 warps x 16)
constexpr int CP_BK = 64;   // reduction elements per pipeline stage
constexpr int CP_THREADS = 128;

template <int DC>
__global__ void __launch_bounds__(CP_THREADS)
compress_kernel(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ W,
                const float* __restrict__ bias, __nv_bfloat16* __restrict__ dst, int rows, int rows_per_seq,
                int d_in, int kslice, int64_t seq_stride, RowMap map) {
    constexpr int CH = CP_BK / 8;  // 16-byte chunks per smem row
    extern __shared__ uint4 smem[];
    uint4* sX[2] = {smem, smem + CP_BM * CH};
    uint4* sW[2] = {smem + 2 * CP_BM * CH, smem + 2 * CP_BM * CH + DC * CH};

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row0 = blockIdx.x * CP_BM;
    const int split = blockIdx.y;
    const int k_begin = split * kslice;
    const int nk = kslice / CP_BK;

    auto load_stage = [&](int st, int kk) {
        const int kofs = k_begin + kk * CP_BK;
        for (int i = tid; i < CP_BM * CH; i += CP_THREADS) {
            int r = i / CH, c = i % CH;
            int gr = row0 + r;
            bool ok = gr < rows;
            const __nv_bfloat16* src = X + (size_t)(ok ? gr : 0) * d_in + kofs + c * 8;
            cp_async16(&sX[st][swz<CH>(r, c)], src, ok ? 16 : 0);
        }
        for (int i = tid; i < DC * CH; i += CP_THREADS) {
            int r = i / CH, c = i % CH;
            cp_async16(&sW[st][swz<CH>(r, c)], W + (size_t)r * d_in + kofs + c * 8);
        }
        cp_async_commit();
    };

    float acc[DC / 8][4];
#pragma unroll
    for (int i = 0; i < DC / 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    load_stage(0, 0);
    for (int kk = 0; kk < nk; ++kk) {
        if (kk + 1 < nk) {
            load_stage((kk + 1) & 1, kk + 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const uint4* tx = sX[kk & 1];
        const uint4* tw = sW[kk & 1];
#pragma unroll
        for (int ks = 0; ks < CP_BK / 16; ++ks) {
            uint32_t a[4];
            load_a_frag<CH>(a, tx, warp * 16, ks * 2, lane);
#pragma unroll
            for (int nb = 0; nb < DC / 16; ++nb) {
                uint32_t b[4];
                load_b_frag_nk<CH>(b, tw, nb * 16, ks * 2, lane);
                mma_bf16_16816(acc[2 * nb], a, b[0], b[1]);
                mma_bf16_16816(acc[2 * nb + 1], a, b[2], b[3]);
            }
        }
        __syncthreads();
    }

    // fp32 partial tile -> this CTA's shared memory
    float* sPart = reinterpret_cast<float*>(smem + 2 * (CP_BM + DC) * CH);   // [CP_BM][DC]
    {
        const int r = warp * 16 + (lane >> 2);
#pragma unroll
        for (int nb = 0; nb < DC / 8; ++nb) {
            int col = nb * 8 + (lane & 3) * 2;
            *reinterpret_cast<float2*>(sPart + r * DC + col) = make_float2(acc[nb][0], acc[nb][1]);
            *reinterpret_cast<float2*>(sPart + (r + 8) * DC + col) = make_float2(acc[nb][2], acc[nb][3]);
        }
    }
    // The CTAs of a cluster hold the split-K partials of one row tile.  Each CTA sums a
    // band of rows over all of them through distributed shared memory, in split order (so
    // the result does not depend on timing), adds the bias and rounds to bf16.
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();
    const int nsplit = gridDim.y;
    const int band = CP_BM / nsplit;                  // rows reduced by this CTA
    constexpr int PER_ROW = DC / 4;
    for (int i = tid; i < band * PER_ROW; i += CP_THREADS) {
        const int lr = split * band + i / PER_ROW, c4 = (i % PER_ROW) * 4;
        const int row = row0 + lr;
        if (row >= rows) continue;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sp = 0; sp < nsplit; ++sp) {
            const float4 v = *reinterpret_cast<const float4*>(cluster.map_shared_rank(sPart, sp) + lr * DC + c4);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        if (bias) {
            s.x += bias[c4]; s.y += bias[c4 + 1]; s.z += bias[c4 + 2]; s.w += bias[c4 + 3];
        }
        const int b = row / rows_per_seq, ii = row % rows_per_seq;
        __nv_bfloat16* o = dst + ((int64_t)b * seq_stride + map.row0[b] + ii) * DC + c4;
        *reinterpret_cast<uint2*>(o) = make_uint2(pack_bf16(s.x, s.y), pack_bf16(s.z, s.w));
    }
    cluster.sync();    // shared memory stays alive until every remote read is done
}

template <int DC>
static cudaError_t launch_compress_t(esa_ctx* ctx, const __nv_bfloat16* X, int rows, int rows_per_seq,
                                     int d_in, const __nv_bfloat16* W, const float* bias,
                                     __nv_bfloat16* dst, int64_t seq_stride, const RowMap& map,
                                     cudaStream_t st) {
    const int row_tiles = (rows + CP_BM - 1) / CP_BM;
    const int nk_total = d_in / CP_BK;
    // split the reduction over a cluster of up to 8 CTAs while that still adds CTAs usefully
    int nsplit = 1;
    while (nsplit < 8 && (nk_total % (nsplit * 2)) == 0 && row_tiles * nsplit < 2 * ctx->num_sms) nsplit *= 2;
    const int kslice = d_in / nsplit;
    constexpr int smem = 2 * (CP_BM + DC) * (CP_BK / 8) * 16 + CP_BM * DC * 4;
    cudaError_t e = cudaFuncSetAttribute(compress_kernel<DC>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(row_tiles, nsplit);
    cfg.blockDim = dim3(CP_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = nsplit;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ProfScope prof(ctx, KC_COMPRESS_MMA, st);
    e = cudaLaunchKernelEx(&cfg, compress_kernel<DC>, X, W, bias, dst, rows, rows_per_seq, d_in, kslice,
                           seq_stride, map);
    ctx->launches += 1;
    return e;
}

cudaError_t launch_compress(esa_ctx* ctx, const __nv_bfloat16* X, int B, int rows_per_seq, int d_in,
                            const __nv_bfloat16* W, const float* bias, __nv_bfloat16* dst,
                            int64_t dst_seq_stride, const RowMap& map, cudaStream_t st) {
    const int rows = B * rows_per_seq;
    switch (ctx->dc) {
        case 32: return launch_compress_t<32>(ctx, X, rows, rows_per_seq, d_in, W, bias, dst, dst_seq_stride, map, st);
        case 64: return launch_compress_t<64>(ctx, X, rows, rows_per_seq, d_in, W, bias, dst, dst_seq_stride, map, st);
        case 128: return launch_compress_t<128>(ctx, X, rows, rows_per_seq, d_in, W, bias, dst, dst_seq_stride, map, st);
    }
    return cudaErrorInvalidValue;
}

// ---------------------------------------------------------------------------
// Eq. 5 for a handful of rows (decode: one new token per sequence).  A GEMM tile would be
// almost empty, so this is a GEMV: one CTA per output feature c.  Its threads split row c of W
// into 16-byte chunks (one or two per thread, every load in flight at once: the kernel is a
// single round trip to L2), form the partial dot products with every input row, and reduce
// them through shuffles and shared memory.  fp32 accumulation, bias, one bf16 rounding.
// ---------------------------------------------------------------------------
constexpr int GEMV_ROWS = 8;        // input rows per pass
constexpr int GEMV_THREADS = 256;

__global__ void __launch_bounds__(GEMV_THREADS)
compress_gemv_kernel(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ W,
                     const float* __restrict__ bias, __nv_bfloat16* __restrict__ dst, int rows, int rows_per_seq,
                     int d_in, int dc, int64_t dst_seq_stride, RowMap map, uint32_t* zero_words, int zero_count,
                     uint32_t* zero2_words, int zero2_count) {
    __shared__ float red[GEMV_THREADS / 32][GEMV_ROWS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int c = blockIdx.x;                              // output feature of this CTA
    const int r0 = blockIdx.y * GEMV_ROWS;                 // first input row of this pass
    pdl_wait();
    pdl_launch_dependents();
    if (zero_words && blockIdx.x == 0 && blockIdx.y == 0)
        for (int i = tid; i < zero_count; i += GEMV_THREADS) zero_words[i] = 0u;
    if (zero2_words && blockIdx.y == 0)
        for (int i = blockIdx.x * GEMV_THREADS + tid; i < zero2_count; i += gridDim.x * GEMV_THREADS) zero2_words[i] = 0u;
    const int nr = min(GEMV_ROWS, rows - r0);
    float acc[GEMV_ROWS];
#pragma unroll
    for (int r = 0; r < GEMV_ROWS; ++r) acc[r] = 0.f;
    const uint4* wrow = reinterpret_cast<const uint4*>(W + (int64_t)c * d_in);
    const int chunks = d_in / 8;
#pragma unroll 2
    for (int ch = tid; ch < chunks; ch += GEMV_THREADS) {
        const uint4 wv = __ldg(wrow + ch);
        uint4 xv[GEMV_ROWS];
#pragma unroll
        for (int r = 0; r < GEMV_ROWS; ++r)
            xv[r] = __ldg(reinterpret_cast<const uint4*>(X + (int64_t)(r0 + min(r, nr - 1)) * d_in) + ch);
        const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&wv);
        float2 wf[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) wf[i] = __bfloat1622float2(w2[i]);
#pragma unroll
        for (int r = 0; r < GEMV_ROWS; ++r) {
            const __nv_bfloat162* x2 = reinterpret_cast<const __nv_bfloat162*>(&xv[r]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 xf = __bfloat1622float2(x2[i]);
                acc[r] = fmaf(wf[i].x, xf.x, acc[r]);
                acc[r] = fmaf(wf[i].y, xf.y, acc[r]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < GEMV_ROWS; ++r) {
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], o);
        if (lane == 0) red[warp][r] = acc[r];
    }
    __syncthreads();
    if (tid < nr) {
        float sum = bias ? bias[c] : 0.f;
#pragma unroll
        for (int w = 0; w < GEMV_THREADS / 32; ++w) sum += red[w][tid];
        const int row = r0 + tid, b = row / rows_per_seq, i = row % rows_per_seq;
        dst[((int64_t)b * dst_seq_stride + map.row0[b] + i) * dc + c] = __float2bfloat16_rn(sum);
    }
}

cudaError_t launch_compress_gemv(esa_ctx* ctx, const __nv_bfloat16* X, int B, int rows_per_seq, int d_in,
                                 const __nv_bfloat16* W, const float* bias, __nv_bfloat16* dst,
                                 int64_t dst_seq_stride, const RowMap& map, uint32_t* zero_words, int zero_count,
                                 uint32_t* zero2_words, int zero2_count, cudaStream_t st) {
    const int rows = B * rows_per_seq;
    if (rows > kCompressGemvRows || d_in % 8 != 0) return cudaErrorNotSupported;
    const dim3 grid(ctx->dc, (rows + GEMV_ROWS - 1) / GEMV_ROWS);
    ProfScope prof(ctx, KC_COMPRESS_GEMV, st);
    cudaError_t e = launch_pdl(compress_gemv_kernel, grid, dim3(GEMV_THREADS), 0, st, X, W, bias, dst, rows,
                               rows_per_seq, d_in, ctx->dc, dst_seq_stride, map, zero_words, zero_count, zero2_words,
                               zero2_count);
    ctx->launches += 1;
    return e;
}

// ---------------------------------------------------------------------------
// K/V cache append: rows of the chunk copied into the caller's caches.
// ---------------------------------------------------------------------------
__global__ void append_kv_kernel(const uint4* __restrict__ K_new, const uint4* __restrict__ V_new,
                                 uint4* __restrict__ K_cache, uint4* __restrict__ V_cache, int n_new,
                                 int row_chunks, int64_t max_tokens, RowMap map) {
    const int b = blockIdx.y;
    const int64_t per_seq = (int64_t)n_new * row_chunks;
    pdl_wait();                 // the previous step's attention may still be reading the caches
    pdl_launch_dependents();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < per_seq;
         i += (int64_t)gridDim.x * blockDim.x) {
        int64_t src = (int64_t)b * per_seq + i;
        int64_t dst = ((int64_t)b * max_tokens + map.row0[b]) * row_chunks + i;
        K_cache[dst] = K_new[src];
        V_cache[dst] = V_new[src];
    }
}

cudaError_t launch_append_kv(esa_ctx* ctx, int B, const __nv_bfloat16* K_new, const __nv_bfloat16* V_new,
                             int n_new, __nv_bfloat16* K_cache, __nv_bfloat16* V_cache,
                             const RowMap& map, cudaStream_t st) {
    const int row_chunks = ctx->dG / 8;
    const int64_t per_seq = (int64_t)n_new * row_chunks;
    int gx = (int)((per_seq + 255) / 256);
    if (gx > 4 * ctx->num_sms) gx = 4 * ctx->num_sms;
    if (gx < 1) gx = 1;
    ProfScope prof(ctx, KC_APPEND_KV, st);
    cudaError_t e = launch_pdl(append_kv_kernel, dim3(gx, B), dim3(256), 0, st,
                               reinterpret_cast<const uint4*>(K_new), reinterpret_cast<const uint4*>(V_new),
                               reinterpret_cast<uint4*>(K_cache), reinterpret_cast<uint4*>(V_cache), n_new, row_chunks,
                               ctx->cfg.max_tokens, map);
    ctx->launches += 1;
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace esa
