// What a trainer-side batch still needs after the features: cepstra (the MFCC
// baseline of the paper's Table 1 is a DCT of log-mel energies), per-utterance mean
// and variance of every feature, and an ordering of utterances by length for
// padded batches (Section 2.2).
#include <algorithm>
#include <numeric>
#include <vector>

#include "common.cuh"

namespace {

// c_i = s_i sum_m x[m] cos(pi i (m + 1/2) / M), s_0 = sqrt(1/M), s_i = sqrt(2/M): orthonormal DCT-II
__global__ void __launch_bounds__(256)
mfcc_kernel(const float *__restrict__ feats, const int *__restrict__ counts, int M, int n_cep,
            int T_max, float pad_v, float *__restrict__ out) {
    extern __shared__ float basis[];                 // [n_cep][M]
    const int utt = blockIdx.y, tid = threadIdx.x;
    constexpr int FT = 16;
    const int t0 = blockIdx.x * FT;
    const int rows = min(FT, T_max - t0);
    if (rows <= 0) return;
    for (int i = tid; i < n_cep * M; i += 256) {
        const int c = i / M, m = i - c * M;
        const float s = c == 0 ? rsqrtf((float)M) : sqrtf(2.f / (float)M);
        basis[i] = s * cospif((float)c * ((float)m + 0.5f) / (float)M);
    }
    __syncthreads();
    const int T = min(max(counts[utt], 0), T_max);
    for (int i = tid; i < rows * n_cep; i += 256) {
        const int f = i / n_cep, c = i - f * n_cep, t = t0 + f;
        float v = pad_v;
        if (t < T) {
            const float *x = feats + ((int64_t)utt * T_max + t) * M;
            const float *bz = basis + c * M;
            float acc = 0.f;
            for (int m = 0; m < M; ++m) acc = fmaf(x[m], bz[m], acc);
            v = acc;
        }
        out[((int64_t)utt * T_max + t) * n_cep + c] = v;
    }
}

// One CTA per utterance; sums in double, so 6000 frames lose nothing.
__global__ void __launch_bounds__(256)
mean_var_kernel(const float *__restrict__ feats, const int *__restrict__ counts, int D, int T_max,
                float *__restrict__ mean, float *__restrict__ var) {
    __shared__ double s1[256], s2[256];
    const int utt = blockIdx.x, tid = threadIdx.x;
    const int T = min(max(counts[utt], 0), T_max);
    const int lanes = 256 / D > 0 ? 256 / D : 1;     // frame slices that work side by side
    for (int d0 = 0; d0 < D; d0 += 256) {
        const int d = d0 + (D >= 256 ? tid : tid % D);
        const int slice = D >= 256 ? 0 : tid / D;
        double a = 0.0, b = 0.0;
        if (d < D && slice < lanes) {
            for (int t = slice; t < T; t += lanes) {
                const double x = feats[((int64_t)utt * T_max + t) * D + d];
                a += x;
                b += x * x;
            }
        }
        s1[tid] = a;
        s2[tid] = b;
        __syncthreads();
        if (d < D && slice == 0) {
            for (int j = 1; j < lanes; ++j) {
                a += s1[tid + j * D];
                b += s2[tid + j * D];
            }
            const double mu = T > 0 ? a / T : 0.0;
            const double vv = T > 0 ? b / T - mu * mu : 0.0;
            mean[(int64_t)utt * D + d] = (float)mu;
            var[(int64_t)utt * D + d] = (float)(vv > 0.0 ? vv : 0.0);
        }
        __syncthreads();
    }
}

}  // namespace

extern "C" int feat_mfcc(AugCtx *ctx, const float *feats_dev, const int *counts_dev, int B, int T_max,
                         int n_cep, float *mfcc_dev) {
    if (!ctx || B < 0) return AUG_EINVAL;
    if (B > ctx->cfg.max_batch) return AUG_ECAP;
    if (B == 0) return AUG_OK;
    const int M = ctx->cfg.n_mel;
    if (!feats_dev || !counts_dev || !mfcc_dev || T_max <= 0 || n_cep < 1 || n_cep > M) return AUG_EINVAL;
    const size_t smem = sizeof(float) * (size_t)n_cep * M;
    if (smem > 96 * 1024) return AUG_ECAP;
    AUG_CUDA_OK(cudaFuncSetAttribute(mfcc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid((T_max + 15) / 16, B);
    mfcc_kernel<<<grid, 256, smem, ctx->stream>>>(feats_dev, counts_dev, M, n_cep, T_max,
                                                  ctx->cfg.pad_value, mfcc_dev);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

extern "C" int feat_mean_var(AugCtx *ctx, const float *feats_dev, const int *counts_dev, int B,
                             int T_max, int D, float *mean_dev, float *var_dev) {
    if (!ctx || B < 0) return AUG_EINVAL;
    if (B > ctx->cfg.max_batch) return AUG_ECAP;
    if (B == 0) return AUG_OK;
    if (!feats_dev || !counts_dev || !mean_dev || !var_dev || T_max <= 0 || D < 1) return AUG_EINVAL;
    mean_var_kernel<<<B, 256, 0, ctx->stream>>>(feats_dev, counts_dev, D, T_max, mean_dev, var_dev);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

extern "C" int aug_bucket_by_length(const int *lengths_host, int B, int batch, int *perm_host,
                                    int *batch_max_host) {
    if (B < 0 || batch < 1 || (B > 0 && (!lengths_host || !perm_host))) return AUG_EINVAL;
    std::vector<int> idx(B);
    std::iota(idx.begin(), idx.end(), 0);
    std::stable_sort(idx.begin(), idx.end(),
                     [&](int a, int b) { return lengths_host[a] < lengths_host[b]; });
    for (int i = 0; i < B; ++i) perm_host[i] = idx[i];
    if (batch_max_host)
        for (int g = 0; g * batch < B; ++g) {
            const int last = std::min(B, (g + 1) * batch) - 1;     // longest of a sorted group
            batch_max_host[g] = lengths_host[idx[last]];
        }
    return AUG_OK;
}
