// Step 2: reverberation by partitioned FFT overlap convolution, noise mixing.
//
// The impulse response is cut into partitions of CONV_BLK taps whose spectra are
// computed once per batch (rir_spectra_kernel).  One CTA then produces one block
// of CONV_BLK output samples: Y_b = sum_p X_{b-p} H_p, where X_j is the spectrum of
// the 2*CONV_BLK input samples that end with block j.  Taking each input block
// together with its predecessor is the overlap-add tail sum moved to the input
// side, so output blocks never exchange data.  All noise sources are summed in
// the frequency domain: two inverse transforms per block whatever their number.
//
// Two routes, same arithmetic:
//   one partition   convolve_fused_kernel: transform the input segment, multiply,
//                   inverse-transform, all in one CTA; nothing but y_s and v is stored.
//   more partitions block_spectra_kernel stores every X_j once; spectral_convolve_kernel
//                   reads the P spectra a block needs (mostly from L2), multiply-
//                   accumulates in registers and inverse-transforms.
//
// A real transform of F points is a complex transform of F/2 points on (even, odd)
// sample pairs followed by the usual split; thread t owns the bin pairs
// (k, F/2-k), k = t + 256 q.  Spectra are stored as F/2 complex numbers with the two
// real bins (0 and F/2) packed into slot 0.
#include "common.cuh"
#include "fft.cuh"

namespace {

using namespace augfft;
constexpr int N2 = aug::CONV_N2;      // 4096 complex points
constexpr int BLK = aug::CONV_BLK;
constexpr int CT = 256;               // threads per CTA
constexpr int E = N2 / CT;            // 16 points per thread: three radix-16 passes
constexpr int NQ = N2 / 2 / CT;       // 8 bin pairs per thread
constexpr int SM_POINTS = padded_points(N2);
#ifndef CONV_MINB
#define CONV_MINB 3                  // CTAs per SM the register budget is set for
#endif

__device__ __forceinline__ void fft4096_from_regs(float2 (*v)[E], float2 *s, int t,
                                                  const float2 *__restrict__ tw) {
    pass_from_regs<N2, E, 16, 1>(v, s, t, tw);
    __syncthreads();
    pass<N2, E, 16, 16, 1>(s, t, tw, CtaSync());
    pass<N2, E, 16, 256, 16>(s, t, tw, CtaSync());
}

__device__ __forceinline__ void fft4096_in_place(float2 *s, int t, const float2 *__restrict__ tw) {
    pass<N2, E, 16, 1, 0>(s, t, tw, CtaSync());
    pass<N2, E, 16, 16, 1>(s, t, tw, CtaSync());
    pass<N2, E, 16, 256, 16>(s, t, tw, CtaSync());
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

// The pair a thread owns for k = t + CT q, read from a finished transform in `sm`:
//   k != 0:  a = X[k],            b = X[N2-k]
//   k == 0:  a = (X[0], X[N2])    b = X[N2/2]      (X[0], X[N2] are real)
__device__ __forceinline__ void spectrum_pair(const float2 *sm, const float2 *__restrict__ tw, int k,
                                              float2 &a, float2 &b) {
    const float2 zk = sm[pad0(k)], zm = sm[pad0((N2 - k) & (N2 - 1))];
    const float2 w = __ldg(&tw[tw_index(aug::CONV_F, k)]);
    float2 xk, xm;
    real_split(zk, zm, w, xk, xm);
    if (k == 0) {
        const float2 zh = sm[pad0(N2 / 2)];
        a = make_float2(xk.x, xm.x);
        b = make_float2(zh.x, -zh.y);
    } else {
        a = xk;
        b = xm;
    }
}
// Slots of that pair in a stored spectrum.
__device__ __forceinline__ int slot_a(int k) { return k; }
__device__ __forceinline__ int slot_b(int k) { return k == 0 ? N2 / 2 : N2 - k; }

__device__ __forceinline__ void mac_pair(float2 &acc_a, float2 &acc_b, float2 a, float2 b, float2 ha,
                                         float2 hb, int k) {
    if (k == 0) {
        acc_a.x = fmaf(a.x, ha.x, acc_a.x);
        acc_a.y = fmaf(a.y, ha.y, acc_a.y);
    } else {
        acc_a = cadd(acc_a, cmul(a, ha));
    }
    acc_b = cadd(acc_b, cmul(b, hb));
}

// 2*BLK input samples starting at `base` as 16 (even, odd) pairs per thread in the
// order the first FFT pass wants them.  Speech reads x[i]; a noise source reads
// its stretch of the bank end to end (x[i mod nlen]).  Outside [0, N): zero.
__device__ __forceinline__ void load_segment(float2 (*v)[E], const float *__restrict__ x, bool looped,
                                             int nlen, int base, int N, int t) {
    if (!looped) {
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int i0 = base + 2 * (t + CT * r);
            float2 z = make_float2(0.f, 0.f);
            if (i0 >= 0) {
                if (i0 + 1 < N) z = *reinterpret_cast<const float2 *>(x + i0);
                else if (i0 < N) z.x = x[i0];
            }
            v[0][r] = z;
        }
        return;
    }
    // Looped source: one division for the first sample, then the position advances
    // by 2*CT (mod nlen) from one pair to the next.
    const int first = base + 2 * t;
    const int step = (2 * CT) % nlen;
    int m = first >= 0 ? first % nlen : (nlen - (-first) % nlen) % nlen;
#pragma unroll
    for (int r = 0; r < E; ++r) {
        const int i0 = first + 2 * CT * r;
        float2 z = make_float2(0.f, 0.f);
        if (i0 >= 0) {
            if (i0 < N) z.x = x[m];
            if (i0 + 1 < N) z.y = x[m + 1 == nlen ? 0 : m + 1];
        }
        v[0][r] = z;
        m += step;
        if (m >= nlen) m -= nlen;
    }
}

// Source s of an utterance: pointer to its samples, loop length; false if the row's
// noise stretch is unusable (reported once through the status word).
__device__ __forceinline__ bool source_of(const AugUttParams &row, int s, const float *speech_row,
                                          const float *bank, int64_t bank_len, const float *&x,
                                          int &nlen) {
    if (s == 0) {
        x = speech_row;
        nlen = 1;
        return true;
    }
    const int64_t off = row.noise_offset[s - 1];
    nlen = row.noise_len[s - 1];
    if (nlen <= 0 || off < 0 || off + nlen > bank_len || bank == nullptr) return false;
    x = bank + off;
    return true;
}

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

// Accumulated block spectrum -> CONV_BLK output samples at dst, plus their energy.
// The half-size spectrum is rebuilt with real and imaginary parts swapped, which
// turns the forward transform into the (unnormalised) inverse; the scale 1/F sits
// in the stored partition spectra.  The second half of the 2*BLK outputs is kept.
__device__ __forceinline__ void finish_block(const float2 (*acc)[2], float2 *sm,
                                             const float2 *__restrict__ tw, int t, float *dst,
                                             int n_left, double *energy_slot, float *red) {
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        const int k = t + CT * q;
        const float2 yk = acc[q][0], ym = acc[q][1];
        if (k == 0) {
            // yk = (Y[0], Y[N2]) real pair; ym = Y[N2/2]
            sm[pad0(0)] = make_float2(yk.x - yk.y, yk.x + yk.y);
            sm[pad0(N2 / 2)] = make_float2(-2.f * ym.y, 2.f * ym.x);
        } else {
            const float2 w = __ldg(&tw[tw_index(aug::CONV_F, k)]);
            // Z[k] = (Yk + conj Ym) + i conj(W)(Yk - conj Ym)
            const float2 a = make_float2(yk.x + ym.x, yk.y - ym.y);
            const float2 d = make_float2(yk.x - ym.x, yk.y + ym.y);
            const float2 e = cmul(make_float2(w.y, w.x), d);       // i conj(W) = (w.y, w.x)
            const float2 zk = make_float2(a.x + e.x, a.y + e.y);
            // Z[N2-k] = (Ym + conj Yk) - i W (Ym - conj Yk)
            const float2 e2 = cmul(make_float2(-w.y, w.x), make_float2(-d.x, d.y));   // i W = (-w.y, w.x)
            const float2 zm = make_float2(a.x - e2.x, -a.y - e2.y);
            sm[pad0(k)] = make_float2(zk.y, zk.x);
            sm[pad0(N2 - k)] = make_float2(zm.y, zm.x);
        }
    }
    __syncthreads();
    fft4096_in_place(sm, t, tw);
    float e2sum = 0.f;
#pragma unroll
    for (int r = 0; r < BLK / 2 / CT; ++r) {
        const int n = t + CT * r;                       // pair index within the block
        const float2 z = sm[pad0(N2 / 2 + n)];          // second half; swapped back here
        const float y0 = z.y, y1 = z.x;
        if (2 * n + 1 < n_left) {
            *reinterpret_cast<float2 *>(dst + 2 * n) = make_float2(y0, y1);
            e2sum += y0 * y0 + y1 * y1;
        } else if (2 * n < n_left) {
            dst[2 * n] = y0;
            e2sum += y0 * y0;
        }
    }
    const float tot = block_sum(e2sum, red, t);
    if (t == 0) atomicAdd(energy_slot, (double)tot);
    __syncthreads();
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

    float2 v[1][E];
#pragma unroll
    for (int r = 0; r < E; ++r) {
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
        float2 a, b;
        spectrum_pair(sm, tw, k, a, b);
        out[slot_a(k)] = make_float2(a.x * scale, a.y * scale);
        out[slot_b(k)] = make_float2(b.x * scale, b.y * scale);
    }
}

// ---------------------------------------------------------------- one partition: fused
__global__ void __launch_bounds__(CT, CONV_MINB)
convolve_fused_kernel(const float *__restrict__ speech, int64_t stride,
                      const int *__restrict__ lengths, const float *__restrict__ bank,
                      int64_t bank_len, const AugUttParams *__restrict__ table, int S_max, int P,
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
    const int n_out = n_src > 1 ? 2 : (n_src == 1 ? 1 : 0);

    for (int o = 0; o < n_out; ++o) {
        float2 acc[NQ][2];
#pragma unroll
        for (int q = 0; q < NQ; ++q) acc[q][0] = acc[q][1] = make_float2(0.f, 0.f);
        const int s_lo = o ? 1 : 0, s_hi = o ? n_src : 1;
        for (int s = s_lo; s < s_hi; ++s) {
            const float *x;
            int nlen;
            if (!source_of(row, s, speech + (int64_t)utt * stride, bank, bank_len, x, nlen)) {
                if (t == 0 && b == 0 && atomicCAS(&status[0], -1, utt) == -1) status[1] = aug::R_NOISE;
                continue;
            }
            for (int p = 0; p < P && p <= b; ++p) {
                float2 v[1][E];
                load_segment(v, x, s != 0, nlen, (b - p - 1) * BLK, N, t);
                fft4096_from_regs(v, sm, t, tw);
                const float2 *H = hspec + (((int64_t)utt * S_max + s) * P + p) * N2;
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const int k = t + CT * q;
                    float2 xa, xb;
                    spectrum_pair(sm, tw, k, xa, xb);
                    mac_pair(acc[q][0], acc[q][1], xa, xb, __ldg(&H[slot_a(k)]), __ldg(&H[slot_b(k)]), k);
                }
                __syncthreads();   // sm is overwritten by the next transform
            }
        }
        float *dst = (o ? vv : ys) + (int64_t)utt * ws_stride + (int64_t)b * BLK;
        finish_block(acc, sm, tw, t, dst, N - b * BLK, &energy[2 * utt + o], red);
    }
    if (n_src <= 1) {
        // no noise: v is defined as silence
        float *dst = vv + (int64_t)utt * ws_stride + (int64_t)b * BLK;
        for (int i = t; i < BLK && b * BLK + i < N; i += CT) dst[i] = 0.f;
    }
}

// ---------------------------------------------------------------- several partitions
// Spectrum of every 2*BLK input segment of every source, stored once.
__global__ void __launch_bounds__(CT, CONV_MINB)
block_spectra_kernel(const float *__restrict__ speech, int64_t stride,
                     const int *__restrict__ lengths, const float *__restrict__ bank,
                     int64_t bank_len, const AugUttParams *__restrict__ table, int S_max,
                     const float2 *__restrict__ tw, float2 *__restrict__ xspec, int nblk_cap,
                     int *status, int n_cap) {
    extern __shared__ __align__(16) float2 sm[];
    const int b = blockIdx.x, s = blockIdx.y, utt = blockIdx.z, t = threadIdx.x;
    const int N = min(max(lengths[utt], 0), n_cap);
    if ((int64_t)b * BLK >= N) return;
    const AugUttParams &row = table[utt];
    if (row.n_src < 1 || row.n_src > S_max || s >= row.n_src) return;
    const float *x;
    int nlen;
    if (!source_of(row, s, speech + (int64_t)utt * stride, bank, bank_len, x, nlen)) {
        if (t == 0 && b == 0 && atomicCAS(&status[0], -1, utt) == -1) status[1] = aug::R_NOISE;
        return;
    }
    float2 v[1][E];
    load_segment(v, x, s != 0, nlen, (b - 1) * BLK, N, t);
    fft4096_from_regs(v, sm, t, tw);
    float2 *out = xspec + (((int64_t)utt * S_max + s) * nblk_cap + b) * N2;
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        const int k = t + CT * q;
        float2 a, bb;
        spectrum_pair(sm, tw, k, a, bb);
        out[slot_a(k)] = a;
        out[slot_b(k)] = bb;
    }
}

__global__ void __launch_bounds__(CT, CONV_MINB)
spectral_convolve_kernel(const int *__restrict__ lengths, const float *__restrict__ bank,
                         int64_t bank_len, const AugUttParams *__restrict__ table, int S_max, int P,
                         const float2 *__restrict__ hspec, const float2 *__restrict__ xspec,
                         int nblk_cap, const float2 *__restrict__ tw, float *__restrict__ ys,
                         float *__restrict__ vv, int64_t ws_stride, double *__restrict__ energy,
                         int n_cap) {
    extern __shared__ __align__(16) float2 sm[];
    __shared__ float red[CT / 32];
    const int b = blockIdx.x, utt = blockIdx.y, t = threadIdx.x;
    const int N = min(max(lengths[utt], 0), n_cap);
    if ((int64_t)b * BLK >= N) return;
    const AugUttParams &row = table[utt];
    int n_src = row.n_src;
    if (n_src < 1 || n_src > S_max) n_src = 0;
    const int n_out = n_src > 1 ? 2 : (n_src == 1 ? 1 : 0);

    for (int o = 0; o < n_out; ++o) {
        float2 acc[NQ][2];
#pragma unroll
        for (int q = 0; q < NQ; ++q) acc[q][0] = acc[q][1] = make_float2(0.f, 0.f);
        const int s_lo = o ? 1 : 0, s_hi = o ? n_src : 1;
        for (int s = s_lo; s < s_hi; ++s) {
            const float *x;
            int nlen;
            if (!source_of(row, s, nullptr, bank, bank_len, x, nlen)) continue;   // no spectra stored
            const float2 *Hs = hspec + ((int64_t)utt * S_max + s) * P * N2;
            const float2 *Xs = xspec + ((int64_t)utt * S_max + s) * nblk_cap * N2;
            for (int p = 0; p < P && p <= b; ++p) {
                const float2 *H = Hs + (int64_t)p * N2;
                const float2 *X = Xs + (int64_t)(b - p) * N2;
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const int k = t + CT * q;
                    const int ia = slot_a(k), ib = slot_b(k);
                    mac_pair(acc[q][0], acc[q][1], __ldg(&X[ia]), __ldg(&X[ib]), __ldg(&H[ia]),
                             __ldg(&H[ib]), k);
                }
            }
        }
        float *dst = (o ? vv : ys) + (int64_t)utt * ws_stride + (int64_t)b * BLK;
        finish_block(acc, sm, tw, t, dst, N - b * BLK, &energy[2 * utt + o], red);
    }
    if (n_src <= 1) {
        float *dst = vv + (int64_t)utt * ws_stride + (int64_t)b * BLK;
        for (int i = t; i < BLK && b * BLK + i < N; i += CT) dst[i] = 0.f;
    }
}

// ---------------------------------------------------------------- mixing
// g = sqrt(sum y_s^2 / (sum v^2 10^(snr/10))), 0 without noise or with a silent side:
// once per utterance, in fp64, after the convolution has finished the two sums.
__global__ void __launch_bounds__(256)
snr_gain_kernel(const double *__restrict__ energy, const AugUttParams *__restrict__ table, int B,
                float *__restrict__ gain) {
    const int utt = blockIdx.x * 256 + threadIdx.x;
    if (utt >= B) return;
    const double es = energy[2 * utt], ev = energy[2 * utt + 1];
    float g = 0.f;
    if (table[utt].n_src > 1 && es > 0.0 && ev > 0.0)
        g = (float)sqrt(es / (ev * pow(10.0, (double)table[utt].snr_db / 10.0)));
    gain[utt] = g;
}

__global__ void __launch_bounds__(256)
mix_kernel(const float *__restrict__ ys, const float *__restrict__ vv, int64_t ws_stride,
           const float *__restrict__ gain, const int *__restrict__ lengths,
           float *__restrict__ out, int64_t out_stride, int n_cap) {
    const int utt = blockIdx.y;
    const int N = min(max(lengths[utt], 0), n_cap);
    const int i = (blockIdx.x * 256 + threadIdx.x) * 4;
    if (i >= N) return;
    const float g = gain[utt];
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

constexpr size_t FFT_SMEM = sizeof(float2) * SM_POINTS;

}  // namespace

int launch_rir_spectra(AugCtx *ctx, const float *rir, const AugUttParams *table, int B,
                       cudaStream_t st) {
    const AugConfig &c = ctx->cfg;
    dim3 grid(ctx->n_part, c.max_sources, B);
    rir_spectra_kernel<<<grid, CT, FFT_SMEM, st>>>(rir, table, c.max_sources, c.rir_taps,
                                                            ctx->n_part, ctx->tw, ctx->hspec);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

static bool stored_route(const AugCtx *ctx) { return ctx->n_part > 1 && ctx->xspec != nullptr; }

int launch_convolve_prepare(AugCtx *ctx, const float *speech, int64_t stride, const int *lengths,
                            const float *bank, int64_t bank_len, const AugUttParams *table, int B,
                            int max_len) {
    const AugConfig &c = ctx->cfg;
    if (max_len <= 0) return AUG_OK;
    AUG_CUDA_OK(cudaMemsetAsync(ctx->energy, 0, sizeof(double) * 2 * (size_t)B, ctx->stream));
    if (!stored_route(ctx)) return AUG_OK;
    const int nblk = (max_len + BLK - 1) / BLK;
    dim3 grid_x(nblk, c.max_sources, B);
    block_spectra_kernel<<<grid_x, CT, FFT_SMEM, ctx->stream>>>(
        speech, stride, lengths, bank, bank_len, table, c.max_sources, ctx->tw, ctx->xspec,
        ctx->nblk_cap, ctx->status, max_len);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

int launch_convolve_finish(AugCtx *ctx, const float *speech, int64_t stride, const int *lengths,
                           const float *bank, int64_t bank_len, const AugUttParams *table, int B,
                           int max_len) {
    const AugConfig &c = ctx->cfg;
    if (max_len <= 0) return AUG_OK;
    const int nblk = (max_len + BLK - 1) / BLK;
    dim3 grid(nblk, B);
    if (!stored_route(ctx)) {
        convolve_fused_kernel<<<grid, CT, FFT_SMEM, ctx->stream>>>(
            speech, stride, lengths, bank, bank_len, table, c.max_sources, ctx->n_part, ctx->hspec,
            ctx->tw, ctx->ys, ctx->vv, ctx->ws_stride, ctx->energy, ctx->status, max_len);
    } else {
        spectral_convolve_kernel<<<grid, CT, FFT_SMEM, ctx->stream>>>(
            lengths, bank, bank_len, table, c.max_sources, ctx->n_part, ctx->hspec, ctx->xspec,
            ctx->nblk_cap, ctx->tw, ctx->ys, ctx->vv, ctx->ws_stride, ctx->energy, max_len);
    }
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    snr_gain_kernel<<<(B + 255) / 256, 256, 0, ctx->stream>>>(ctx->energy, table, B, ctx->gain);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

int launch_mix(AugCtx *ctx, const int *lengths, const AugUttParams *table, int B, int max_len,
               float *wave_out, int64_t out_stride) {
    if (max_len <= 0) return AUG_OK;
    dim3 grid((max_len + 1023) / 1024, B);
    mix_kernel<<<grid, 256, 0, ctx->stream>>>(ctx->ys, ctx->vv, ctx->ws_stride, ctx->gain, lengths,
                                              wave_out, out_stride, max_len);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}
