// K/V cache resident in host memory (the paper's single-GPU mode, appendix "Model Loading": the
// full K/V cache is offloaded to the CPU, the compressed keys stay on the GPU, and every attention
// computation brings a small number of keys and values onto the GPU).
//
// gather_kv_kernel copies the rows of the attended list I u M_k u L u C, in list order, from the
// host-resident caches (pinned memory mapped into the device's address space: the loads cross
// PCIe) into compact device staging caches; the attention kernels then run on the staged rows,
// which form a plain contiguous list (every staged row before the chunk is "initial", nothing is
// selected), so they compute exactly what they compute on device-resident caches.
#include "esa_internal.h"

namespace esa {

namespace {

struct GatherParams {
    const uint4* K_host;      // [B, max_tokens, HG * D / 8] (16-byte units)
    const uint4* V_host;
    uint4* K_stage;           // [B, stage_rows, HG * D / 8]
    uint4* V_stage;
    const int32_t* idx;       // [B, top_k]
    const int32_t* n_sel;     // [B]
    int* status;
    int64_t max_tokens;
    int64_t stage_rows;
    int row_units;            // 16-byte units per row
    int l_C, top_k;
    SeqMeta meta;
};

// One warp per list row and iteration; a row is row_units 16-byte units, read with 16-byte loads
// (whole 512-byte segments per warp instruction: the widest request a device-side read of host
// memory makes).
__global__ void __launch_bounds__(256) gather_kv_kernel(GatherParams p) {
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int n_warps = (gridDim.x * blockDim.x) >> 5;
    pdl_wait();                    // the selection comes from the preceding kernel
    pdl_launch_dependents();
    const int t = p.meta.t[b], i_end = p.meta.i_end[b], m_end = p.meta.m_end[b];
    int n_sel = p.n_sel[b];
    n_sel = max(0, min(n_sel, min(p.top_k, m_end - i_end)));
    const int n_glob = i_end + n_sel;
    const int n_att = n_glob + (t - m_end) + p.l_C;
    int bad = 0;
    for (int j0 = warp * 4; j0 < n_att; j0 += n_warps * 4) {
        // four rows per round, their loads in flight together
        int pos[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = j0 + u;
            int q = -1;
            if (j < n_att) {
                if (j < i_end) q = j;
                else if (j < n_glob) q = clamp_selected(__ldg(p.idx + (int64_t)b * p.top_k + (j - i_end)), i_end, m_end, bad);
                else q = m_end + (j - n_glob);
            }
            pos[u] = q;
        }
        for (int c0 = 0; c0 < p.row_units; c0 += 32) {
            const int c = c0 + lane;
            uint4 kv[4], vv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (pos[u] >= 0 && c < p.row_units) {
                    const int64_t src = ((int64_t)b * p.max_tokens + pos[u]) * p.row_units + c;
                    kv[u] = p.K_host[src];
                    vv[u] = p.V_host[src];
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (pos[u] >= 0 && c < p.row_units) {
                    const int64_t dst = ((int64_t)b * p.stage_rows + j0 + u) * p.row_units + c;
                    p.K_stage[dst] = kv[u];
                    p.V_stage[dst] = vv[u];
                }
            }
        }
    }
    if (bad) atomicExch(p.status, kStatusBadIndex);
}

}  // namespace

// Stages the attended rows of every sequence and returns, in staged_meta, the partition under which
// the staged rows are a plain contiguous list (t = rows before the chunk, all of them "initial").
cudaError_t launch_gather_kv(esa_ctx* ctx, int B, int l_C, const void* K_host, const void* V_host, const SeqMeta& meta,
                             const int32_t* idx, const int32_t* n_sel, void* K_stage, void* V_stage, int64_t stage_rows,
                             cudaStream_t st) {
    GatherParams p;
    p.K_host = (const uint4*)K_host; p.V_host = (const uint4*)V_host;
    p.K_stage = (uint4*)K_stage; p.V_stage = (uint4*)V_stage;
    p.idx = idx; p.n_sel = n_sel; p.status = ctx->status;
    p.max_tokens = ctx->cfg.max_tokens; p.stage_rows = stage_rows; p.row_units = ctx->dG / 8;
    p.l_C = l_C; p.top_k = ctx->cfg.top_k; p.meta = meta;
    int gx = 4 * ctx->num_sms / B;
    if (gx < 1) gx = 1;
    ProfScope prof(ctx, KC_GATHER_KV, st);
    cudaError_t e = launch_pdl(gather_kv_kernel, dim3(gx, B), dim3(256), 0, st, p);
    ctx->launches += 1;
    return e;
}

}  // namespace esa
