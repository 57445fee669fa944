// Eq. 7: fitting the two linear compressors f_q(q) = W_q q + b_q and f_k(k) = W_k k + b_k so that
// f_q(q_c) . f_k(k_m) reproduces the full-dimension score q_c k_m^T (Eq. 3) of every query-key pair
// of a batch (mean squared error over the n x n pairs), with Adam.  An offline, per-layer step
// (Section 4.1: learning rate 5e-4, batches of 128 pairs, 10 epochs over 50k pairs): a few small
// products per step, bound by launch latency and fp32 arithmetic, kept in fp32 throughout so that
// thousands of steps stay close to a double-precision run.
//
// One step (n pairs; Q [n, H, d] and K [n, H_G, d] bf16 on the device):
//   Qf = heads of each GQA group summed            T  = Qf K^T            (Eq. 3 for all pairs)
//   A  = Q W_q^T + b_q      Bm = K W_k^T + b_k     E  = A Bm^T - T        loss = mean(E^2)
//   dP = 2 E / n^2          dA = dP Bm             dBm = dP^T A
//   dW_q = dA^T Q   db_q = column sums of dA       dW_k = dBm^T K   db_k = column sums of dBm
//   Adam update of W_q, b_q, W_k, b_k
#include <cmath>
#include <new>

#include "esa_internal.h"

struct esa_fit {
    int device;
    int H, HG, d, dc, dH, dG, n;
    float lr, beta1, beta2, eps;
    int64_t step;
    char* base;
    size_t n_params;              // dc*dH + dc + dc*dG + dc
    float* params;                // [Wq | bq | Wk | bk]
    float* grads;                 // same layout
    float* m1;                    // Adam first moments
    float* m2;                    // Adam second moments
    float *Qf, *T, *A, *Bm, *dP, *dA, *dBm;
    float* part;                  // partial sums of split reductions
    float* loss_acc;              // one float
    int64_t launches;
};

namespace esa {
namespace {

constexpr int GT = 64;            // output tile of the generic product kernel
constexpr int GK = 16;

__device__ __forceinline__ float ldf(const float* p, int64_t i) { return p[i]; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p, int64_t i) { return __bfloat162float(p[i]); }

// C[m, n] = sum_k A(m, k) B(n, k) + bias[n] - sub[m, n], fp32 accumulation in the order of k.
// A(m, k) = A[m * sam + k * sak], B(n, k) = B[n * sbn + k * sbk]: any of the four transpose
// combinations by strides.  64 x 64 output tile per CTA, 4 x 4 outputs per thread.  A long reduction
// is cut into gridDim.z ranges of kslice columns: CTA z then writes its raw partial sums to
// C + z * M * N, and fit_reduce_kernel adds the partials in the order of z (so the result does not
// depend on scheduling) and applies bias and sub.
template <typename TA, typename TB>
__global__ void __launch_bounds__(256) fit_gemm_kernel(const TA* __restrict__ A, int64_t sam, int64_t sak, const TB* __restrict__ B,
                                                       int64_t sbn, int64_t sbk, float* __restrict__ C, int M, int N, int K,
                                                       int kslice, const float* __restrict__ bias, const float* __restrict__ sub) {
    __shared__ float sA[GK][GT + 1];
    __shared__ float sB[GK][GT + 1];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * GT, n0 = blockIdx.x * GT;
    const int tm = (tid / 16) * 4, tn = (tid % 16) * 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    const int k_begin = blockIdx.z * kslice;
    if (gridDim.z > 1) {
        K = min(K, k_begin + kslice);
        C += (int64_t)blockIdx.z * M * N;
    }
    for (int k0 = k_begin; k0 < K; k0 += GK) {
        for (int e = tid; e < GT * GK; e += 256) {
            // the faster-varying index follows the operand's unit stride
            const int r = sak == 1 ? e / GK : e % GT, kk = sak == 1 ? e % GK : e / GT;
            sA[kk][r] = (m0 + r < M && k0 + kk < K) ? ldf(A, (int64_t)(m0 + r) * sam + (int64_t)(k0 + kk) * sak) : 0.f;
            const int r2 = sbk == 1 ? e / GK : e % GT, k2 = sbk == 1 ? e % GK : e / GT;
            sB[k2][r2] = (n0 + r2 < N && k0 + k2 < K) ? ldf(B, (int64_t)(n0 + r2) * sbn + (int64_t)(k0 + k2) * sbk) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < GK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = sA[kk][tm + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = sB[kk][tn + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int m = m0 + tm + i, n = n0 + tn + j;
            if (m < M && n < N) {
                float v = acc[i][j];
                if (bias) v += bias[n];
                if (sub) v -= sub[(int64_t)m * N + n];
                C[(int64_t)m * N + n] = v;
            }
        }
}

// C[e] = sum over z (in order) of part[z][e] + bias[e % N] - sub[e]
__global__ void fit_reduce_kernel(const float* __restrict__ part, int splits, float* __restrict__ C, int M, int N,
                                  const float* __restrict__ bias, const float* __restrict__ sub) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= M * N) return;
    float v = 0.f;
    for (int z = 0; z < splits; ++z) v += part[(int64_t)z * M * N + e];
    if (bias) v += bias[e % N];
    if (sub) v -= sub[e];
    C[e] = v;
}

// Qf[c, g, i] = sum over the heads h of group g of Q[c, h, i] (fp32)
__global__ void fit_fold_kernel(const __nv_bfloat16* __restrict__ Q, float* __restrict__ Qf, int n, int H, int HG, int d) {
    const int G = H / HG;
    const int64_t total = (int64_t)n * HG * d;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int i = e % d, g = (e / d) % HG;
        const int64_t c = e / ((int64_t)d * HG);
        float s = 0.f;
        for (int h = 0; h < G; ++h) s += __bfloat162float(Q[(c * H + g * G + h) * d + i]);
        Qf[e] = s;
    }
}

// loss += sum E^2 / count (one atomic per CTA);  dP = 2 E / count
__global__ void fit_loss_kernel(const float* __restrict__ E, float* __restrict__ dP, float* __restrict__ loss, int count) {
    __shared__ float red[32];
    float s = 0.f;
    const float inv = 1.f / (float)count;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < count; e += gridDim.x * blockDim.x) {
        const float v = E[e];
        s += v * v;
        dP[e] = 2.f * v * inv;
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x < 32) {
        s = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (threadIdx.x == 0) atomicAdd(loss, s * inv);
    }
}

// column sums of X [n, dc] -> out [dc]
__global__ void fit_colsum_kernel(const float* __restrict__ X, float* __restrict__ out, int n, int dc) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= dc) return;
    float s = 0.f;
    for (int r = 0; r < n; ++r) s += X[(int64_t)r * dc + j];
    out[j] = s;
}

__global__ void fit_adam_kernel(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ m1, float* __restrict__ m2,
                                size_t count, float lr, float beta1, float beta2, float eps, float c1, float c2) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < count; e += (size_t)gridDim.x * blockDim.x) {
        const float gr = g[e];
        const float m = beta1 * m1[e] + (1.f - beta1) * gr;
        const float v = beta2 * m2[e] + (1.f - beta2) * gr * gr;
        m1[e] = m;
        m2[e] = v;
        p[e] -= lr * (m / c1) / (sqrtf(v / c2) + eps);
    }
}

// `part`: scratch for split reductions (kFitMaxSplit * M * N floats), or null to reduce in one CTA per tile
constexpr int kFitMaxSplit = 32;
template <typename TA, typename TB>
int gemm(cudaStream_t st, const TA* A, int64_t sam, int64_t sak, const TB* B, int64_t sbn, int64_t sbk, float* C, int M, int N, int K,
         const float* bias = nullptr, const float* sub = nullptr, float* part = nullptr) {
    const dim3 tiles((N + GT - 1) / GT, (M + GT - 1) / GT);
    int splits = 1;
    if (part) {
        while (splits < kFitMaxSplit && (int)(tiles.x * tiles.y) * splits < 128 && K / (splits * 2) >= 4 * GK) splits *= 2;
    }
    if (splits == 1) {
        fit_gemm_kernel<TA, TB><<<tiles, 256, 0, st>>>(A, sam, sak, B, sbn, sbk, C, M, N, K, K, bias, sub);
        return 1;
    }
    const int kslice = ((K + splits - 1) / splits + GK - 1) / GK * GK;
    fit_gemm_kernel<TA, TB><<<dim3(tiles.x, tiles.y, splits), 256, 0, st>>>(A, sam, sak, B, sbn, sbk, part, M, N, K, kslice, nullptr, nullptr);
    fit_reduce_kernel<<<(M * N + 255) / 256, 256, 0, st>>>(part, splits, C, M, N, bias, sub);
    return 2;
}

}  // namespace
}  // namespace esa

using namespace esa;

extern "C" {

esa_status esa_fit_create(const esa_config* cfg, int32_t batch, float lr, esa_fit** out) {
    if (!out) return ESA_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cfg || batch <= 0 || batch > 4096 || !(lr > 0.f)) return ESA_ERR_INVALID_ARG;
    if (cfg->n_q_heads <= 0 || cfg->n_kv_heads <= 0 || cfg->n_q_heads % cfg->n_kv_heads || cfg->head_dim <= 0 || cfg->d_c <= 0)
        return ESA_ERR_SHAPE;
    esa_fit* f = new (std::nothrow) esa_fit();
    if (!f) return ESA_ERR_INVALID_ARG;
    f->H = cfg->n_q_heads; f->HG = cfg->n_kv_heads; f->d = cfg->head_dim; f->dc = cfg->d_c;
    f->dH = f->H * f->d; f->dG = f->HG * f->d; f->n = batch;
    f->lr = lr; f->beta1 = 0.9f; f->beta2 = 0.999f; f->eps = 1e-8f;
    f->step = 0;
    f->launches = 0;
    f->n_params = (size_t)f->dc * f->dH + f->dc + (size_t)f->dc * f->dG + f->dc;
    const size_t n = batch, dc = f->dc;
    const size_t part_floats = 32 * (n * n > n * dc ? n * n : n * dc);
    const size_t floats = 4 * f->n_params + n * f->dG + 2 * n * n + 4 * n * dc + part_floats + 64;
    if (cudaGetDevice(&f->device) != cudaSuccess || cudaMalloc(&f->base, floats * sizeof(float)) != cudaSuccess) {
        cudaGetLastError();
        delete f;
        return ESA_ERR_CUDA;
    }
    float* p = reinterpret_cast<float*>(f->base);
    f->params = p; p += f->n_params;
    f->grads = p; p += f->n_params;
    f->m1 = p; p += f->n_params;
    f->m2 = p; p += f->n_params;
    f->Qf = p; p += n * f->dG;
    f->T = p; p += n * n;
    f->dP = p; p += n * n;
    f->A = p; p += n * dc;
    f->Bm = p; p += n * dc;
    f->dA = p; p += n * dc;
    f->dBm = p; p += n * dc;
    f->part = p; p += part_floats;
    f->loss_acc = p;
    if (cudaMemset(f->base, 0, floats * sizeof(float)) != cudaSuccess) {
        cudaFree(f->base);
        delete f;
        return ESA_ERR_CUDA;
    }
    *out = f;
    return ESA_OK;
}

esa_status esa_fit_destroy(esa_fit* f) {
    if (!f) return ESA_ERR_INVALID_ARG;
    cudaError_t e = cudaFree(f->base);
    delete f;
    return e == cudaSuccess ? ESA_OK : ESA_ERR_CUDA;
}

static void fit_offsets(const esa_fit* f, size_t* wq, size_t* bq, size_t* wk, size_t* bk) {
    *wq = 0;
    *bq = (size_t)f->dc * f->dH;
    *wk = *bq + f->dc;
    *bk = *wk + (size_t)f->dc * f->dG;
}

esa_status esa_fit_set_weights(esa_fit* f, const float* Wq, const float* bq, const float* Wk, const float* bk) {
    if (!f || !Wq || !Wk) return ESA_ERR_INVALID_ARG;
    size_t owq, obq, owk, obk;
    fit_offsets(f, &owq, &obq, &owk, &obk);
    // parameters, and a fresh optimiser state
    if (cudaMemset(f->params, 0, 4 * f->n_params * sizeof(float)) != cudaSuccess) return ESA_ERR_CUDA;
    if (cudaMemcpy(f->params + owq, Wq, sizeof(float) * f->dc * f->dH, cudaMemcpyHostToDevice) != cudaSuccess) return ESA_ERR_CUDA;
    if (cudaMemcpy(f->params + owk, Wk, sizeof(float) * f->dc * f->dG, cudaMemcpyHostToDevice) != cudaSuccess) return ESA_ERR_CUDA;
    if (bq && cudaMemcpy(f->params + obq, bq, sizeof(float) * f->dc, cudaMemcpyHostToDevice) != cudaSuccess) return ESA_ERR_CUDA;
    if (bk && cudaMemcpy(f->params + obk, bk, sizeof(float) * f->dc, cudaMemcpyHostToDevice) != cudaSuccess) return ESA_ERR_CUDA;
    f->step = 0;
    return ESA_OK;
}

esa_status esa_fit_get_weights(esa_fit* f, float* Wq, float* bq, float* Wk, float* bk) {
    if (!f || !Wq || !bq || !Wk || !bk) return ESA_ERR_INVALID_ARG;
    size_t owq, obq, owk, obk;
    fit_offsets(f, &owq, &obq, &owk, &obk);
    if (cudaDeviceSynchronize() != cudaSuccess) return ESA_ERR_CUDA;
    if (cudaMemcpy(Wq, f->params + owq, sizeof(float) * f->dc * f->dH, cudaMemcpyDeviceToHost) != cudaSuccess) return ESA_ERR_CUDA;
    if (cudaMemcpy(bq, f->params + obq, sizeof(float) * f->dc, cudaMemcpyDeviceToHost) != cudaSuccess) return ESA_ERR_CUDA;
    if (cudaMemcpy(Wk, f->params + owk, sizeof(float) * f->dc * f->dG, cudaMemcpyDeviceToHost) != cudaSuccess) return ESA_ERR_CUDA;
    if (cudaMemcpy(bk, f->params + obk, sizeof(float) * f->dc, cudaMemcpyDeviceToHost) != cudaSuccess) return ESA_ERR_CUDA;
    return ESA_OK;
}

esa_status esa_fit_step_async(esa_fit* f, const void* Q_batch, const void* K_batch, int32_t n, float* loss_out, void* stream) {
    if (!f || !Q_batch || !K_batch || n <= 0) return ESA_ERR_INVALID_ARG;
    if (n > f->n) return ESA_ERR_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    const __nv_bfloat16* Q = (const __nv_bfloat16*)Q_batch;
    const __nv_bfloat16* K = (const __nv_bfloat16*)K_batch;
    size_t owq, obq, owk, obk;
    fit_offsets(f, &owq, &obq, &owk, &obk);
    float *Wq = f->params + owq, *bq = f->params + obq, *Wk = f->params + owk, *bk = f->params + obk;
    const int dc = f->dc, dH = f->dH, dG = f->dG;
    // targets (Eq. 3 for every pair)
    fit_fold_kernel<<<(unsigned)(((int64_t)n * dG + 255) / 256), 256, 0, st>>>(Q, f->Qf, n, f->H, f->HG, f->d);
    int launches = 5;                                  // fold, loss, two column sums, Adam
    launches += gemm(st, f->Qf, (int64_t)dG, 1, K, (int64_t)dG, 1, f->T, n, n, dG, nullptr, nullptr, f->part);
    // forward
    launches += gemm(st, Q, (int64_t)dH, 1, Wq, (int64_t)dH, 1, f->A, n, dc, dH, bq, nullptr, f->part);
    launches += gemm(st, K, (int64_t)dG, 1, Wk, (int64_t)dG, 1, f->Bm, n, dc, dG, bk, nullptr, f->part);
    launches += gemm(st, f->A, (int64_t)dc, 1, f->Bm, (int64_t)dc, 1, f->dP, n, n, dc, nullptr, f->T, f->part);      // E = A Bm^T - T (in dP's buffer)
    if (cudaMemsetAsync(f->loss_acc, 0, sizeof(float), st) != cudaSuccess) return ESA_ERR_CUDA;
    fit_loss_kernel<<<32, 256, 0, st>>>(f->dP, f->dP, f->loss_acc, n * n);
    // backward
    launches += gemm(st, f->dP, (int64_t)n, 1, f->Bm, 1, (int64_t)dc, f->dA, n, dc, n);                      // dA[c, j] = sum_m dP[c, m] Bm[m, j]
    launches += gemm(st, f->dP, 1, (int64_t)n, f->A, 1, (int64_t)dc, f->dBm, n, dc, n);                      // dBm[m, j] = sum_c dP[c, m] A[c, j]
    launches += gemm(st, f->dA, 1, (int64_t)dc, Q, 1, (int64_t)dH, f->grads + owq, dc, dH, n);               // dWq[j, i] = sum_c dA[c, j] Q[c, i]
    launches += gemm(st, f->dBm, 1, (int64_t)dc, K, 1, (int64_t)dG, f->grads + owk, dc, dG, n);
    fit_colsum_kernel<<<(dc + 127) / 128, 128, 0, st>>>(f->dA, f->grads + obq, n, dc);
    fit_colsum_kernel<<<(dc + 127) / 128, 128, 0, st>>>(f->dBm, f->grads + obk, n, dc);
    // Adam
    f->step += 1;
    const float c1 = 1.f - std::pow(f->beta1, (float)f->step), c2 = 1.f - std::pow(f->beta2, (float)f->step);
    fit_adam_kernel<<<256, 256, 0, st>>>(f->params, f->grads, f->m1, f->m2, f->n_params, f->lr, f->beta1, f->beta2, f->eps, c1, c2);
    f->launches += launches;
    if (loss_out && cudaMemcpyAsync(loss_out, f->loss_acc, sizeof(float), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return ESA_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? ESA_OK : ESA_ERR_CUDA;
}

int64_t esa_fit_launch_count(const esa_fit* f) { return f ? f->launches : -1; }

}  // extern "C"
