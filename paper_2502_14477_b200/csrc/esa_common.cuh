// Device-side helpers shared by the ESA kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace esa {

constexpr int kMaxBatch = 64;

// Per-sequence scalars of one call, passed by value in the kernel parameters.
// t = tokens preceding the chunk; [i_end, m_end) = middle tokens (Section 3.1).
struct SeqMeta {
    int t[kMaxBatch];
    int i_end[kMaxBatch];
    int m_end[kMaxBatch];
};

// ---------------------------------------------------------------------------
// order-preserving map fp32 -> uint32 (larger float <=> larger key); -0 is
// folded into +0 first so equal scores get equal keys.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t f32_to_key(float f) {
    uint32_t u = __float_as_uint(f + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_f32(uint32_t k) {
    uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(u);
}

// ---------------------------------------------------------------------------
// shared-memory tiles: rows of ROW_CHUNKS 16-byte chunks, chunk index XOR-swizzled
// with the row so that ldmatrix (8 rows x 16 B) and 16-byte row stores are
// bank-conflict free.
// ---------------------------------------------------------------------------
template <int ROW_CHUNKS>
__device__ __forceinline__ int swz(int row, int chunk) {
    if constexpr (ROW_CHUNKS >= 8) {
        return row * ROW_CHUNKS + (chunk ^ (row & 7));
    } else if constexpr (ROW_CHUNKS == 4) {
        return row * ROW_CHUNKS + (chunk ^ ((row >> 1) & 3));
    } else {
        return row * ROW_CHUNKS + chunk;
    }
}

// A selected position handed to the attention must lie in M = [i_end, m_end).  One that does not
// (a stale or corrupted index buffer) is replaced by the nearest position of M, so that no row
// outside the caches is ever read, and `bad` is raised; the caller records ESA_ERR_INDEX once.
constexpr int kStatusBadIndex = 8;
__device__ __forceinline__ int clamp_selected(int q, int i_end, int m_end, int& bad) {
    if ((unsigned)(q - i_end) >= (unsigned)(m_end - i_end)) {
        bad = 1;
        q = q < i_end ? i_end : m_end - 1;
    }
    return q;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte async copy global -> shared; src_bytes = 0 zero-fills the destination.
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, int src_bytes = 16) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(smem_u32(smem)), "l"(gmem),
                 "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_u32(smem)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_u32(smem)));
}

// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                               uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may
// start while its predecessor in the stream is still draining.  pdl_wait() returns once the predecessor
// has completed and its writes are visible (a no-op for an ordinary launch); everything a kernel
// reads from or writes to global memory comes after it.  pdl_launch_dependents() lets the successor's
// CTAs take the SMs this grid frees at its tail.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

// 2^x, hardware approximation (ex2.approx: 2^-inf = +0)
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// A-operand fragment (16 rows x 16 k) of a K-major tile: row0 = first row, kc = first
// 16-byte chunk of the k-step.
template <int ROW_CHUNKS>
__device__ __forceinline__ void load_a_frag(uint32_t (&a)[4], const uint4* tile, int row0, int kc,
                                            int lane) {
    int r = row0 + (lane & 7) + ((lane >> 3) & 1) * 8;
    int c = kc + (lane >> 4);
    ldmatrix_x4(a, tile + swz<ROW_CHUNKS>(r, c));
}
// B-operand fragments for two adjacent 8-wide n-blocks from a tile stored [n][k]
// (k contiguous): b[0],b[1] -> n-block n0, b[2],b[3] -> n-block n0+8.
template <int ROW_CHUNKS>
__device__ __forceinline__ void load_b_frag_nk(uint32_t (&b)[4], const uint4* tile, int n0, int kc,
                                               int lane) {
    int r = n0 + (lane & 7) + ((lane >> 4) & 1) * 8;
    int c = kc + ((lane >> 3) & 1);
    ldmatrix_x4(b, tile + swz<ROW_CHUNKS>(r, c));
}
// B-operand fragments from a tile stored [k][n] (n contiguous): k0 = first of 16 k rows,
// nc = 16-byte chunk holding n-block n0 (8 columns); b[0],b[1] -> chunk nc, b[2],b[3] -> nc+1.
template <int ROW_CHUNKS>
__device__ __forceinline__ void load_b_frag_kn(uint32_t (&b)[4], const uint4* tile, int k0, int nc,
                                               int lane) {
    int r = k0 + (lane & 7) + ((lane >> 3) & 1) * 8;
    int c = nc + (lane >> 4);
    ldmatrix_x4_trans(b, tile + swz<ROW_CHUNKS>(r, c));
}

}  // namespace esa
