// Step 2: reverberation by partitioned FFT overlap convolution, noise mixing.
//
// The impulse response is cut into partitions of CONV_BLK taps whose spectra are
// computed once per batch (rir_spectra_kernel).  convolve_kernel then produces
// one block of CONV_BLK output samples per CTA: for every source and partition p
// it transforms the 2*CONV_BLK input samples ending at that block shifted back by
// p blocks, multiplies by the partition spectrum and accumulates in registers;
// the previous block's tail is folded in by taking the input segment with its
// predecessor (the overlap-add sum expressed on the input side), so blocks never
// exchange data.  All noise sources are summed in the frequency domain: two
// inverse transforms per block whatever the number of sources.
//
// A real transform of F points is done as a complex transform of F/2 points on
// (even, odd) sample pairs followed by the usual split; thread t owns the bin
// pairs (k, F/2-k), k = t + 512 q, both for the split and for the accumulators.
#include "common.cuh"
#include "fft.cuh"

namespace {

using namespace augfft;
constexpr int N2 = aug::CONV_N2;      // 4096 complex points
constexpr int BLK = aug::CONV_BLK;
constexpr int CT = 512;               // threads per CTA
constexpr int E = N2 / CT;            // 8 points per thread
constexpr int NQ = N2 / 2 / CT;       // 4 bin pairs per thread

__device__ __forceinline__ void fft4096_from_regs(float2 (*v)[8], float2 *s, int t,
                                                  const float2 *__restrict__ tw) {
    pass_from_regs<N2, E, 8, 1>(v, s, t, tw);
    __syncthreads();
    pass<N2, E, 8, 8>(s, t, tw, CtaSync());
    pass<N2, E, 8, 64>(s, t, tw, CtaSync());
    pass<N2, E, 8, 512>(s, t, tw, CtaSync());
}

// Split of the half-size transform Z into the spectrum X of the real signal at the
// bin pair (k, N2-k):  X[k] = Ev + W^k Od,  X[N2-k] = conj(Ev - W^k Od),
// Ev = (Z[k] + conj Z[N2-k])/2, Od = -i (Z[k] - conj Z[N2-k])/2, W = exp(-2 pi i/F).
__device__ __forceinline__ void real_split(float2 zk, float2 zm, float2 w, float2 &xk, float2 &xm) {
    const float2 ev = make_float2(0.5f * (zk.x + zm.x), 0.5f * (zk.y - zm.y));
    const float2 od = make_float2(0.5f * (zk.y + zm.y), -0.5f * (zk.x - zm.x));
    const float2 wo = cmul(w, od);
    xk = make_float2(ev.x + wo.x, ev.y + wo.y);
    xm = make_float2(ev.x - wo.x, -(ev.y - wo.y));
}

// ---------------------------------------------------------------- partition spectra
__global__ void __launch_bounds__(CT)
rir_spectra_kernel(const float *__restrict__ rir, const AugUttParams *__restrict__ table, int S_max,
                   int L, int P, const float2 *__restrict__ tw, float2 *__restrict__ hspec) {
    extern __shared__ __align__(16) float2 sm[];
    const int p = blockIdx.x, s = blockIdx.y, utt = blockIdx.z, t = threadIdx.x;
    const AugUttParams &row = table[utt];
    if (row.n_src < 1 || row.n_src > S_max || s >= row.n_src) return;
    const float scale = (s == 0 ? 1.f : row.noise_weight[s - 1]) / (float)aug::CONV_F;
    const float *h = rir + ((int64_t)utt * S_max + s) * L;
    float2 *out = hspec + (((int64_t)utt * S_max + s) * P + p) * N2;

    float2 v[1][8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const int n = t + CT * r;                 // complex index; taps 2n, 2n+1 of the partition
        const int i0 = p * BLK + 2 * n;
        float2 z = make_float2(0.f, 0.f);
        if (n < BLK / 2) {
            if (i0 < L) z.x = h[i0];
            if (i0 + 1 < L) z.y = h[i0 + 1];
        }
        v[0][r] = z;
    }
    fft4096_from_regs(v, sm, t, tw);
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        const int k = t + CT * q;
        const float2 zk = sm[k], zm = sm[(N2 - k) & (N2 - 1)];
        const float2 w = __ldg(&tw[k * (TW_N / aug::CONV_F)]);
        float2 xk, xm;
        real_split(zk, zm, w, xk, xm);
        if (k == 0) {
            out[0] = make_float2(xk.x * scale, xm.x * scale);   // bins 0 and N2, both real
            const float2 zh = sm[N2 / 2];
            out[N2 / 2] = make_float2(zh.x * scale, -zh.y * scale);
        } else {
            out[k] = make_float2(xk.x * scale, xk.y * scale);
            out[N2 - k] = make_float2(xm.x * scale, xm.y * scale);
        }
    }
}

// ---------------------------------------------------------------- convolution
__device__ __forceinline__ float block_sum(float x, float *red, int t) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    __syncthreads();
    if ((t & 31) == 0) red[t >> 5] = x;
    __syncthreads();
    float tot = 0.f;
    if (t < 32) {
        tot = (t < CT / 32) ? red[t] : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
    }
    return tot;   // valid in warp 0
}

__global__ void __launch_bounds__(CT, 1)
convolve_kernel(const float *__restrict__ speech, int64_t stride, const int *__restrict__ lengths,
                const float *__restrict__ bank, int64_t bank_len,
                const AugUttParams *__restrict__ table, int S_max, int P,
                const float2 *__restrict__ hspec, const float2 *__restrict__ tw,
                float *__restrict__ ys, float *__restrict__ vv, int64_t ws_stride,
                double *__restrict__ energy, int *status, int n_cap) {
    extern __shared__ __align__(16) float2 sm[];
    __shared__ float red[CT / 32];
    const int b = blockIdx.x, utt = blockIdx.y, t = threadIdx.x;
    const int N = min(max(lengths[utt], 0), n_cap);
    if ((int64_t)b * BLK >= N) return;
    const AugUttParams &row = table[utt];
    int n_src = row.n_src;
    if (n_src < 1 || n_src > S_max) n_src = 0;   // rejected row: silence (reported by step 1)

    float2 acc_s[NQ][2], acc_v[NQ][2];
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        acc_s[q][0] = acc_s[q][1] = make_float2(0.f, 0.f);
        acc_v[q][0] = acc_v[q][1] = make_float2(0.f, 0.f);
    }

    for (int s = 0; s < n_src; ++s) {
        const float *x = nullptr;
        int nlen = 1;
        if (s == 0) {
            x = speech + (int64_t)utt * stride;
        } else {
            const int64_t off = row.noise_offset[s - 1];
            nlen = row.noise_len[s - 1];
            if (nlen <= 0 || off < 0 || off + nlen > bank_len || bank == nullptr) {
                if (t == 0 && b == 0 && atomicCAS(&status[0], -1, utt) == -1) status[1] = aug::R_NOISE;
                continue;
            }
            x = bank + off;
        }
        for (int p = 0; p < P; ++p) {
            const int bp = b - p;
            if (bp < 0) break;
            const int base = (bp - 1) * BLK;       // first sample of the 2*BLK segment
            float2 v[1][8];
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const int i0 = base + 2 * (t + CT * r);
                float2 z = make_float2(0.f, 0.f);
                if (s == 0) {
                    if (i0 >= 0 && i0 + 1 < N) {
                        z = *reinterpret_cast<const float2 *>(x + i0);
                    } else if (i0 >= 0 && i0 < N) {
                        z.x = x[i0];
                    }
                } else if (i0 >= 0) {
                    if (i0 < N) z.x = x[i0 % nlen];
                    if (i0 + 1 < N) z.y = x[(i0 + 1) % nlen];
                }
                v[0][r] = z;
            }
            fft4096_from_regs(v, sm, t, tw);
            const float2 *H = hspec + (((int64_t)utt * S_max + s) * P + p) * N2;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int k = t + CT * q;
                const float2 zk = sm[k], zm = sm[(N2 - k) & (N2 - 1)];
                const float2 w = __ldg(&tw[k * (TW_N / aug::CONV_F)]);
                float2 xk, xm;
                real_split(zk, zm, w, xk, xm);
                float2 pk, pm;
                if (k == 0) {
                    const float2 h0 = __ldg(&H[0]);
                    pk = make_float2(xk.x * h0.x, xm.x * h0.y);      // bins 0 and N2 packed
                    const float2 zh = sm[N2 / 2];
                    pm = cmul(make_float2(zh.x, -zh.y), __ldg(&H[N2 / 2]));  // bin N2/2
                } else {
                    pk = cmul(xk, __ldg(&H[k]));
                    pm = cmul(xm, __ldg(&H[N2 - k]));
                }
                if (s == 0) {
                    acc_s[q][0] = cadd(acc_s[q][0], pk);
                    acc_s[q][1] = cadd(acc_s[q][1], pm);
                } else {
                    acc_v[q][0] = cadd(acc_v[q][0], pk);
                    acc_v[q][1] = cadd(acc_v[q][1], pm);
                }
            }
            __syncthreads();   // sm is overwritten by the next transform
        }
    }

    // Inverse transforms: rebuild the half-size spectrum (with real and imaginary
    // parts swapped, which turns the forward transform into the inverse), run it,
    // and keep the second half of the 2*BLK outputs.
    const int n_out = (n_src > 1) ? 2 : 1;
    for (int o = 0; o < n_out; ++o) {
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const int k = t + CT * q;
            const float2 yk = o ? acc_v[q][0] : acc_s[q][0];
            const float2 ym = o ? acc_v[q][1] : acc_s[q][1];
            if (k == 0) {
                // yk = (Y[0], Y[N2]) real pair; ym = Y[N2/2]
                sm[0] = make_float2(yk.x - yk.y, yk.x + yk.y);
                sm[N2 / 2] = make_float2(-2.f * ym.y, 2.f * ym.x);
            } else {
                const float2 w = __ldg(&tw[k * (TW_N / aug::CONV_F)]);
                // Z[k] = (Yk + conj Ym) + i conj(W)(Yk - conj Ym)
                const float2 a = make_float2(yk.x + ym.x, yk.y - ym.y);
                const float2 d = make_float2(yk.x - ym.x, yk.y + ym.y);
                const float2 e = cmul(make_float2(w.y, w.x), d);   // i conj(W) = (w.y, w.x)... see note
                const float2 zk = make_float2(a.x + e.x, a.y + e.y);
                // Z[N2-k] = (Ym + conj Yk) - i W (Ym - conj Yk)
                const float2 a2 = make_float2(a.x, -a.y);
                const float2 d2 = make_float2(-d.x, d.y);
                const float2 e2 = cmul(make_float2(-w.y, w.x), d2);  // i W = (-w.y, w.x)
                const float2 zm = make_float2(a2.x - e2.x, a2.y - e2.y);
                sm[k] = make_float2(zk.y, zk.x);
                sm[N2 - k] = make_float2(zm.y, zm.x);
            }
        }
        __syncthreads();
        pass<N2, E, 8, 1>(sm, t, tw, CtaSync());
        pass<N2, E, 8, 8>(sm, t, tw, CtaSync());
        pass<N2, E, 8, 64>(sm, t, tw, CtaSync());
        pass<N2, E, 8, 512>(sm, t, tw, CtaSync());
        float *dst = (o ? vv : ys) + (int64_t)utt * ws_stride + (int64_t)b * BLK;
        float e2sum = 0.f;
#pragma unroll
        for (int r = 0; r < BLK / 2 / CT; ++r) {
            const int n = t + CT * r;                   // pair index within the block
            const float2 z = sm[N2 / 2 + n];            // second half; swapped back below
            const int i0 = b * BLK + 2 * n;
            const float y0 = z.y, y1 = z.x;
            if (i0 + 1 < N) {
                *reinterpret_cast<float2 *>(dst + 2 * n) = make_float2(y0, y1);
                e2sum += y0 * y0 + y1 * y1;
            } else if (i0 < N) {
                dst[2 * n] = y0;
                e2sum += y0 * y0;
            }
        }
        const float tot = block_sum(e2sum, red, t);
        if (t == 0) atomicAdd(&energy[2 * utt + o], (double)tot);
        __syncthreads();
    }
    if (n_src <= 1) {
        // no noise: v is defined as silence
        float *dst = vv + (int64_t)utt * ws_stride + (int64_t)b * BLK;
        for (int i = t; i < BLK && b * BLK + i < N; i += CT) dst[i] = 0.f;
    }
}

// ---------------------------------------------------------------- mixing
__device__ __forceinline__ float snr_gain(const double *energy, int utt, int n_src, float snr_db) {
    const double es = energy[2 * utt], ev = energy[2 * utt + 1];
    if (n_src <= 1 || !(es > 0.0) || !(ev > 0.0)) return 0.f;
    return (float)sqrt(es / (ev * pow(10.0, (double)snr_db / 10.0)));
}

__global__ void __launch_bounds__(256)
mix_kernel(const float *__restrict__ ys, const float *__restrict__ vv, int64_t ws_stride,
           const double *__restrict__ energy, const int *__restrict__ lengths,
           const AugUttParams *__restrict__ table, float *__restrict__ out, int64_t out_stride,
           int n_cap) {
    const int utt = blockIdx.y;
    const int N = min(max(lengths[utt], 0), n_cap);
    const int i = (blockIdx.x * 256 + threadIdx.x) * 4;
    if (i >= N) return;
    const float g = snr_gain(energy, utt, table[utt].n_src, table[utt].snr_db);
    const float *a = ys + (int64_t)utt * ws_stride + i;
    const float *b = vv + (int64_t)utt * ws_stride + i;
    float *o = out + (int64_t)utt * out_stride + i;
    if (i + 3 < N) {
        const float4 x = *reinterpret_cast<const float4 *>(a);
        const float4 y = *reinterpret_cast<const float4 *>(b);
        *reinterpret_cast<float4 *>(o) =
            make_float4(fmaf(g, y.x, x.x), fmaf(g, y.y, x.y), fmaf(g, y.z, x.z), fmaf(g, y.w, x.w));
    } else {
        for (int j = 0; j < 4 && i + j < N; ++j) o[j] = fmaf(g, b[j], a[j]);
    }
}

}  // namespace

int launch_rir_spectra(AugCtx *ctx, const float *rir, const AugUttParams *table, int B) {
    const AugConfig &c = ctx->cfg;
    const size_t smem = sizeof(float2) * N2;
    AUG_CUDA_OK(cudaFuncSetAttribute(rir_spectra_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem));
    dim3 grid(ctx->n_part, c.max_sources, B);
    rir_spectra_kernel<<<grid, CT, smem, ctx->stream>>>(rir, table, c.max_sources, c.rir_taps,
                                                        ctx->n_part, ctx->tw, ctx->hspec);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

int launch_convolve(AugCtx *ctx, const float *speech, int64_t stride, const int *lengths,
                    const float *bank, int64_t bank_len, const AugUttParams *table, int B,
                    int max_len) {
    const AugConfig &c = ctx->cfg;
    if (max_len <= 0) return AUG_OK;
    const size_t smem = sizeof(float2) * N2;
    AUG_CUDA_OK(cudaFuncSetAttribute(convolve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem));
    AUG_CUDA_OK(cudaMemsetAsync(ctx->energy, 0, sizeof(double) * 2 * (size_t)B, ctx->stream));
    dim3 grid((max_len + BLK - 1) / BLK, B);
    convolve_kernel<<<grid, CT, smem, ctx->stream>>>(speech, stride, lengths, bank, bank_len, table,
                                                     c.max_sources, ctx->n_part, ctx->hspec, ctx->tw,
                                                     ctx->ys, ctx->vv, ctx->ws_stride, ctx->energy,
                                                     ctx->status, max_len);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

int launch_mix(AugCtx *ctx, const int *lengths, const AugUttParams *table, int B, int max_len,
               float *wave_out, int64_t out_stride) {
    if (max_len <= 0) return AUG_OK;
    dim3 grid((max_len + 1023) / 1024, B);
    mix_kernel<<<grid, 256, 0, ctx->stream>>>(ctx->ys, ctx->vv, ctx->ws_stride, ctx->energy, lengths,
                                              table, wave_out, out_stride, max_len);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}
