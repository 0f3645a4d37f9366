// Step 2: reverberation by FFT overlap convolution, noise mixing.
//
// Every route is overlap-save in form: an output block is computed from the input
// segment that ends with it (the block plus the samples before it that the response
// reaches back to), which is the overlap-add tail sum moved to the input side, so
// output blocks never exchange data.  The route is fixed by the response length:
//
//   up to 8192 taps   convolve_fused2_kernel: ONE partition of a 16384-point real
//                     transform, 16384 - taps + 1 outputs per block.  A CTA does the
//                     whole block per source -- forward, multiply, inverse -- and
//                     nothing but y_s and v is stored.  The 8192-point complex
//                     transform of the (even, odd) sample pairs runs as two
//                     4096-point transforms joined by a radix-2 step (second half
//                     of this file).  Several noise sources are summed in the frequency domain
//                     through a small parking area in global memory (one inverse).
//   longer            partitions of CONV_BLK = 4096 taps of an 8192-point transform,
//                     Y_b = sum_p X_{b-p} H_p with X_j the spectrum of the 8192
//                     samples that end with block j: block_spectra_kernel stores
//                     every X_j once; spectral_convolve_kernel reads the P spectra a
//                     block needs (mostly from L2), multiply-accumulates in registers
//                     and inverse-transforms.  Noise sources are summed in the
//                     frequency domain: two inverse transforms per block.
//
// Responses are often shorter than their buffer: behind the last image source's window
// every tap is exactly zero.  The kernels that transform the responses record, per
// utterance, the number of taps up to the last non-zero one (the largest over its
// sources); the fused route then takes 16384 - that + 1 outputs from every block
// instead of 16384 - rir_taps + 1, and the stored-spectra route skips the partitions
// that are zero throughout.  A context sized for long responses sends a batch whose
// responses all end within 8192 taps through the fused route as well: the kernels of
// both routes are launched, look at the batch's largest effective length first, and
// those of the route not taken return at once.  The largest effective length of a batch
// is also copied to the host without waiting for it; while the last value seen says
// "long", the next call launches the stored-spectra kernels alone (they serve any
// length), so a stream of long-response batches pays nothing for the choice.  (Routing
// utterance by utterance was
// measured too: a minority of long CTAs of the fused kernel beside the stored-spectra
// kernels balanced badly.)  The result is the same convolution.
//
// A real transform of F points is a complex transform of F/2 points on (even, odd)
// sample pairs followed by the usual split; in the 8192-point routes thread t owns
// the bin pairs (k, F/2-k), k = t + 256 q.  Spectra are stored as F/2 complex numbers
// with the two real bins (0 and F/2) packed into slot 0; the partition spectra of
// the responses carry the noise weight and the 1/F of the inverse.
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
static_assert(CONV_MINB == aug::PARK_PER_SM, "one parking slot per resident CTA of the fused convolution");

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
    // A segment inside the utterance, and for a looped stretch inside one period of it on
    // 8-byte boundaries, needs no test per pair (the same for the whole CTA).
    if (base >= 0 && base + 2 * BLK <= N) {
        int m0 = base;
        bool plain = !looped;
        if (looped && (nlen & 1) == 0 && (reinterpret_cast<uintptr_t>(x) & 7) == 0) {
            m0 = base % nlen;
            plain = (m0 & 1) == 0 && m0 + 2 * BLK <= nlen;
        }
        if (plain) {
            const float2 *x2 = reinterpret_cast<const float2 *>(x + m0) + t;
#pragma unroll
            for (int r = 0; r < E; ++r) v[0][r] = __ldg(x2 + CT * r);
            return;
        }
    }
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

// Effective length of the responses: (index + 1) of the last non-zero tap, largest over the
// sources of an utterance (leff[utt]) and over the batch (*leff_all); both zeroed before the launch.
__global__ void __launch_bounds__(CT)
rir_length_kernel(const float *__restrict__ rir, const AugUttParams *__restrict__ table, int S_max, int L,
                  int *__restrict__ leff, int *__restrict__ leff_all) {
    __shared__ int red_i[CT / 32];
    const int s = blockIdx.x, utt = blockIdx.y, t = threadIdx.x;
    const AugUttParams &row = table[utt];
    if (row.n_src < 1 || row.n_src > S_max || s >= row.n_src) return;
    const float *h = rir + ((int64_t)utt * S_max + s) * L;
    int last = 0;
    if ((reinterpret_cast<uintptr_t>(h) & 15) == 0) {
        for (int i = 4 * t; i + 3 < L; i += 4 * CT) {
            const float4 z = __ldg(reinterpret_cast<const float4 *>(h + i));
            if (z.x != 0.f) last = i + 1;
            if (z.y != 0.f) last = i + 2;
            if (z.z != 0.f) last = i + 3;
            if (z.w != 0.f) last = i + 4;
        }
        for (int i = (L & ~3) + t; i < L; i += CT)
            if (h[i] != 0.f) last = max(last, i + 1);
    } else {
        for (int i = t; i < L; i += CT)
            if (h[i] != 0.f) last = i + 1;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
    if ((t & 31) == 0) red_i[t >> 5] = last;
    __syncthreads();
    if (t == 0) {
        int m = 0;
        for (int i = 0; i < CT / 32; ++i) m = max(m, red_i[i]);
        if (m > 0) {
            atomicMax(&leff[utt], m);
            atomicMax(leff_all, m);
        }
    }
}

// Which route a batch takes in a context sized for responses of more than 8192 taps.
__device__ __forceinline__ bool takes_fused_route(int leff_batch) { return leff_batch <= 2 * BLK; }

// ---------------------------------------------------------------- partition spectra
__global__ void __launch_bounds__(CT)
rir_spectra_kernel(const float *__restrict__ rir, const AugUttParams *__restrict__ table, int S_max,
                   int L, int P, const float2 *__restrict__ tw, float2 *__restrict__ hspec,
                   const int *__restrict__ leff_all, int always) {
    extern __shared__ __align__(16) float2 sm[];
    const int p = blockIdx.x, s = blockIdx.y, utt = blockIdx.z, t = threadIdx.x;
    if (!always && takes_fused_route(*leff_all)) return;
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

// ---------------------------------------------------------------- several partitions
// Spectrum of every 2*BLK input segment of every source, stored once.
__global__ void __launch_bounds__(CT, CONV_MINB)
block_spectra_kernel(const float *__restrict__ speech, int64_t stride,
                     const int *__restrict__ lengths, const float *__restrict__ bank,
                     int64_t bank_len, const AugUttParams *__restrict__ table, int S_max,
                     const float2 *__restrict__ tw, float2 *__restrict__ xspec, int nblk_cap,
                     int *status, int n_cap, const int *__restrict__ leff_all, int always) {
    extern __shared__ __align__(16) float2 sm[];
    const int b = blockIdx.x, s = blockIdx.y, utt = blockIdx.z, t = threadIdx.x;
    const int N = min(max(lengths[utt], 0), n_cap);
    if ((int64_t)b * BLK >= N || (!always && takes_fused_route(*leff_all))) return;
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
                         int n_cap, const int *__restrict__ leff, const int *__restrict__ leff_all,
                         int always) {
    extern __shared__ __align__(16) float2 sm[];
    __shared__ float red[CT / 32];
    const int b = blockIdx.x, utt = blockIdx.y, t = threadIdx.x;
    // partitions behind the last non-zero tap of every source of this utterance are zero
    const int P_used = min(P, (max(leff[utt], 1) + BLK - 1) / BLK);
    const int N = min(max(lengths[utt], 0), n_cap);
    if ((int64_t)b * BLK >= N || (!always && takes_fused_route(*leff_all))) return;
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
            for (int p = 0; p < P_used && p <= b; ++p) {
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

// ================================================================ 8192-sample blocks
// Impulse responses of 4097..8192 taps fit one partition of a 16384-point real
// transform, so a CTA can do the whole block -- forward, multiply, inverse --
// without any stored spectra.  The 8192-point complex transform of the (even, odd)
// pairs is run as two 4096-point transforms (pairs 0, 2, 4, ... in buffer A, pairs
// 1, 3, 5, ... in buffer B: one 128-bit load feeds one point of each) joined by a
// radix-2 step.  Thread t owns, for k = t + 256 q < 2048, slots k and 4096-k of
// both buffers; from those four numbers it forms bins k, 8192-k, 4096-k and
// 4096+k of the real signal's spectrum, multiplies them with the response's
// bins, and folds the products back into the two half-size inputs of the inverse
// transform -- in place, with no exchange between threads.  Spectra are stored as
// 8192 complex numbers, bins 0 and 8192 (both real) packed into slot 0.
constexpr int BLK2 = 2 * BLK;          // output samples per block
constexpr int F2 = 2 * BLK2;           // real transform size
constexpr int NB2 = F2 / 2;            // complex bins stored per spectrum
constexpr int NQ2 = N2 / 2 / CT;       // slot pairs per thread and buffer

// 2*BLK2 input samples starting at `base`: thread t gets samples
// base + 4 (t + 256 r) + {0,1} as point r of buffer A and + {2,3} as point r of B.
__device__ __forceinline__ void load_segment4(float2 (*va)[E], float2 (*vb)[E],
                                              const float *__restrict__ x, bool looped, int nlen,
                                              int base, int N, int t, const float *xend) {
    // A segment that lies inside the utterance (most do), and for a looped stretch inside one
    // period of it on 16-byte boundaries, needs no test per group: the same for the whole CTA.
    if (base >= 0 && base + F2 <= N) {
        int m0 = base;
        bool plain = !looped;
        if (looped && (nlen & 3) == 0 && (reinterpret_cast<uintptr_t>(x) & 15) == 0) {
            m0 = base % nlen;
            plain = m0 + F2 <= nlen;
        }
        if (plain) {
            const float4 *x4 = reinterpret_cast<const float4 *>(x + m0) + t;
#pragma unroll
            for (int r = 0; r < E; ++r) {
                const float4 z = __ldg(x4 + CT * r);
                va[0][r] = make_float2(z.x, z.y);
                vb[0][r] = make_float2(z.z, z.w);
            }
            return;
        }
    }
    if (!looped) {
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int i0 = base + 4 * (t + CT * r);
            float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i0 >= 0) {
                if (i0 + 3 < N) {
                    z = __ldg(reinterpret_cast<const float4 *>(x + i0));
                } else {
                    if (i0 < N) z.x = x[i0];
                    if (i0 + 1 < N) z.y = x[i0 + 1];
                    if (i0 + 2 < N) z.z = x[i0 + 2];
                }
            }
            va[0][r] = make_float2(z.x, z.y);
            vb[0][r] = make_float2(z.z, z.w);
        }
        return;
    }
    const int first = base + 4 * t;
    const int step = (4 * CT) % nlen;
    int m = first >= 0 ? first % nlen : (nlen - (-first) % nlen) % nlen;
    if ((nlen & 3) == 0 && (reinterpret_cast<uintptr_t>(x) & 15) == 0) {
        // A stretch that starts on a 16-byte boundary and whose length is a multiple
        // of four samples never wraps inside a group of four: one 128-bit load each.
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int i0 = first + 4 * CT * r;
            float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i0 >= 0 && i0 < N) {
                z = __ldg(reinterpret_cast<const float4 *>(x + m));
                if (i0 + 3 >= N) {
                    z.w = 0.f;
                    if (i0 + 2 >= N) z.z = 0.f;
                    if (i0 + 1 >= N) z.y = 0.f;
                }
            }
            va[0][r] = make_float2(z.x, z.y);
            vb[0][r] = make_float2(z.z, z.w);
            m += step;
            if (m >= nlen) m -= nlen;
        }
        return;
    }
    // Any other stretch: a group of four that does not wrap is read as the aligned
    // 128-bit word it starts in and, if it starts a samples into that word, the next
    // word as well (a second round, so that the first loads are all in flight
    // together; neighbouring threads bring that word into L1).  Groups that wrap, end
    // with the utterance or would touch bytes past the bank are read sample by sample.
    const int m0 = m;
    const int room = (int)min((int64_t)0x7fffffff, (int64_t)(xend - x));   // samples from x to the end of the bank
    const int a0 = (int)((reinterpret_cast<uintptr_t>(x) >> 2) & 3);       // where in a 128-bit word x starts
    unsigned amask = 0;                  // 2 bits per group: a, where the second round is needed
#pragma unroll
    for (int r = 0; r < E; ++r) {
        const int i0 = first + 4 * CT * r;
        float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i0 >= 0 && i0 < N) {
            const int a = (a0 + m) & 3;
            if (m + 3 < nlen && i0 + 3 < N && (a == 0 || m - a + 8 <= room)) {
                z = __ldg(reinterpret_cast<const float4 *>(x + (m - a)));
                amask |= (unsigned)a << (2 * r);
            } else {
                int j = m;
                z.x = x[j];
                j = j + 1 == nlen ? 0 : j + 1;
                if (i0 + 1 < N) z.y = x[j];
                j = j + 1 == nlen ? 0 : j + 1;
                if (i0 + 2 < N) z.z = x[j];
                j = j + 1 == nlen ? 0 : j + 1;
                if (i0 + 3 < N) z.w = x[j];
            }
        }
        va[0][r] = make_float2(z.x, z.y);
        vb[0][r] = make_float2(z.z, z.w);
        m += step;
        if (m >= nlen) m -= nlen;
    }
    if (__any_sync(0xffffffffu, amask != 0)) {
        m = m0;
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int a = (int)(amask >> (2 * r)) & 3;
            if (a) {
                const float4 q = __ldg(reinterpret_cast<const float4 *>(x + m - a + 4));
                const float2 lo = va[0][r], hi = vb[0][r];
                // samples a .. a+3 of the eight in (lo, hi, q)
                va[0][r] = a == 1 ? make_float2(lo.y, hi.x) : a == 2 ? hi : make_float2(hi.y, q.x);
                vb[0][r] = a == 1 ? make_float2(hi.y, q.x) : a == 2 ? make_float2(q.x, q.y) : make_float2(q.y, q.z);
            }
            m += step;
            if (m >= nlen) m -= nlen;
            // four second-round loads at a time: more in flight would not fit the registers
            if ((r & 3) == 3) asm volatile("" ::: "memory");
        }
    }
}

// Passes two and three of both half transforms, shared by the forward and the
// inverse direction (a real call: the kernel's instruction footprint matters).
// On entry A is complete and visible and B at most one barrier away from it.
// Returns with B written but not yet synchronised: the caller's barrier finishes it
// (loads that do not depend on the transform go in front of that barrier).
__device__ __noinline__ void fft2x4096_tail(float2 *A, float2 *B, int t, const float2 *__restrict__ tw) {
    pass_pair<N2, E, 16, 16, 1>(A, B, t, tw, CtaSync());
    pass_pair<N2, E, 16, 256, 16>(A, B, t, tw, CtaSync());
}

// Both half transforms of a segment held in registers; on return A and B hold the
// 4096-point transforms of the even and odd pairs, complete and synchronised.
__device__ __forceinline__ void fft2x4096_from_regs(float2 (*va)[E], float2 (*vb)[E], float2 *A,
                                                    float2 *B, int t, const float2 *__restrict__ tw) {
    pass_from_regs<N2, E, 16, 1>(va, A, t, tw);
    pass_from_regs<N2, E, 16, 1>(vb, B, t, tw);
    __syncthreads();
    fft2x4096_tail(A, B, t, tw);
}
// (both variants leave the closing barrier to the caller)

__device__ __forceinline__ void fft2x4096_in_place(float2 *A, float2 *B, int t,
                                                   const float2 *__restrict__ tw) {
    pass_pair<N2, E, 16, 1, 0>(A, B, t, tw, CtaSync());
    fft2x4096_tail(A, B, t, tw);
}

// Inverse of real_split, unnormalised (twice the value): the half-size spectrum
// at the bin pair (k, M-k) from the real signal's bins Y[k], Y[M-k]; W = W_{2M}^k.
__device__ __forceinline__ void real_unsplit(float2 yk, float2 ym, float2 w, float2 &zk, float2 &zm) {
    const float2 a = make_float2(yk.x + ym.x, yk.y - ym.y);          // Yk + conj Ym
    const float2 d = make_float2(yk.x - ym.x, yk.y + ym.y);          // Yk - conj Ym
    const float2 e = cmul(make_float2(w.y, w.x), d);                 // i conj(W) d
    zk = make_float2(a.x + e.x, a.y + e.y);
    const float2 e2 = cmul(make_float2(-w.y, w.x), make_float2(d.x, -d.y));   // i W conj(d)
    zm = make_float2(a.x + e2.x, -a.y + e2.y);
}

// The four bins a thread forms for slot k (1 <= k < 2048) from the two half
// transforms: X[k], X[8192-k], X[4096-k], X[4096+k].
struct Quad {
    float2 k, nk, mk, pk;
};
__device__ __forceinline__ Quad quad_forward(float2 ze_k, float2 ze_m, float2 zo_k, float2 zo_m,
                                             float2 w, float2 u) {
    // radix-2 join: Z[k], Z[k+4096], Z[4096-k], Z[8192-k]
    const float2 t1 = cmul(w, zo_k), t2 = cmul(cconj(w), zo_m);
    const float2 z_k = cadd(ze_k, t1), z_pk = csub(ze_k, t1);
    const float2 z_mk = csub(ze_m, t2), z_nk = cadd(ze_m, t2);
    Quad x;
    real_split(z_k, z_nk, u, x.k, x.nk);
    real_split(z_mk, z_pk, make_float2(-u.y, -u.x), x.mk, x.pk);    // W_F^(4096-k) = -i conj(u)
    return x;
}
// Products back to the inputs of the two half-size inverse transforms, real and
// imaginary parts swapped (the forward code then computes the inverse).
__device__ __forceinline__ void quad_inverse(const Quad &y, float2 w, float2 u, float2 &a_k,
                                             float2 &a_m, float2 &b_k, float2 &b_m) {
    float2 z_k, z_nk, z_mk, z_pk;
    real_unsplit(y.k, y.nk, u, z_k, z_nk);
    real_unsplit(y.mk, y.pk, make_float2(-u.y, -u.x), z_mk, z_pk);
    const float2 s1 = cadd(z_k, z_pk), d1 = cmul(csub(z_k, z_pk), cconj(w));
    const float2 s2 = cadd(z_mk, z_nk), d2 = cmul(csub(z_nk, z_mk), w);   // -(Z[4096-k]-Z[8192-k]) w
    a_k = make_float2(s1.y, s1.x);
    b_k = make_float2(d1.y, d1.x);
    a_m = make_float2(s2.y, s2.x);
    b_m = make_float2(d2.y, d2.x);
}

// Slots 0 and 2048 of both buffers (thread 0): bins 0, 8192 (packed), 4096, 2048, 6144.
struct Edge {
    float2 dc;       // (X[0], X[8192]), both real
    float2 mid;      // X[4096]
    float2 q1, q3;   // X[2048], X[6144]
};
__device__ __forceinline__ Edge edge_forward(float2 ze0, float2 zo0, float2 zeh, float2 zoh, float2 uh) {
    Edge x;
    const float2 z0 = cadd(ze0, zo0), z4 = csub(ze0, zo0);
    x.dc = make_float2(z0.x + z0.y, z0.x - z0.y);
    x.mid = cconj(z4);
    const float2 th = cmul_mi(zoh);                                 // W_8192^2048 = -i
    real_split(cadd(zeh, th), csub(zeh, th), uh, x.q1, x.q3);
    return x;
}
__device__ __forceinline__ void edge_inverse(const Edge &y, float2 uh, float2 &a0, float2 &b0,
                                             float2 &ah, float2 &bh) {
    const float2 z0 = make_float2(y.dc.x + y.dc.y, y.dc.x - y.dc.y);
    const float2 z4 = make_float2(2.f * y.mid.x, -2.f * y.mid.y);
    const float2 s0 = cadd(z0, z4), d0 = csub(z0, z4);
    float2 z2, z6;
    real_unsplit(y.q1, y.q3, uh, z2, z6);
    const float2 sh = cadd(z2, z6), dd = csub(z2, z6);
    const float2 dh = make_float2(-dd.y, dd.x);                     // times conj(-i) = i
    a0 = make_float2(s0.y, s0.x);
    b0 = make_float2(d0.y, d0.x);
    ah = make_float2(sh.y, sh.x);
    bh = make_float2(dh.y, dh.x);
}

// Spectrum of one 16384-sample segment of each impulse response (taps beyond L and
// the whole second half are zero), scaled by the noise weight and 1/F.
__global__ void __launch_bounds__(CT)
rir_spectra2_kernel(const float *__restrict__ rir, const AugUttParams *__restrict__ table, int S_max,
                    int L, const float2 *__restrict__ tw, float2 *__restrict__ hspec, int64_t hs_stride,
                    const int *__restrict__ leff, const int *__restrict__ leff_all, int mixed) {
    extern __shared__ __align__(16) float2 sm[];
    __shared__ int red_i[CT / 32];
    float2 *A = sm, *Bf = sm + SM_POINTS;
    const int s = blockIdx.x, utt = blockIdx.y, t = threadIdx.x;
    // mixed: the lengths are known already (rir_length_kernel) and decide the route; otherwise
    // this kernel reads every tap anyway and records the length on the way
    if (mixed && !takes_fused_route(*leff_all)) return;
    const AugUttParams &row = table[utt];
    if (row.n_src < 1 || row.n_src > S_max || s >= row.n_src) return;
    const float scale = (s == 0 ? 1.f : row.noise_weight[s - 1]) / (float)F2;
    const float *h = rir + ((int64_t)utt * S_max + s) * L;
    float2 *out = hspec + ((int64_t)utt * S_max + s) * hs_stride;
    {
        float2 va[1][E], vb[1][E];
        int last = 0;
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int i0 = 4 * (t + CT * r);
            float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i0 < BLK2) {
                if (i0 < L) z.x = h[i0];
                if (i0 + 1 < L) z.y = h[i0 + 1];
                if (i0 + 2 < L) z.z = h[i0 + 2];
                if (i0 + 3 < L) z.w = h[i0 + 3];
                if (z.x != 0.f) last = i0 + 1;
                if (z.y != 0.f) last = i0 + 2;
                if (z.z != 0.f) last = i0 + 3;
                if (z.w != 0.f) last = i0 + 4;
            }
            va[0][r] = make_float2(z.x, z.y);
            vb[0][r] = make_float2(z.z, z.w);
        }
        if (!mixed) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
            if ((t & 31) == 0) red_i[t >> 5] = last;
            __syncthreads();
            if (t == 0) {
                int m = 0;
                for (int i = 0; i < CT / 32; ++i) m = max(m, red_i[i]);
                if (m > 0) atomicMax(const_cast<int *>(&leff[utt]), m);
            }
        }
        fft2x4096_from_regs(va, vb, A, Bf, t, tw);
        __syncthreads();
    }
#pragma unroll
    for (int q = 0; q < NQ2; ++q) {
        const int k = t + CT * q;
        if (k == 0) {
            const Edge x = edge_forward(A[pad0(0)], Bf[pad0(0)], A[pad0(N2 / 2)], Bf[pad0(N2 / 2)],
                                        __ldg(&tw[tw_index(F2, N2 / 2)]));
            out[0] = make_float2(x.dc.x * scale, x.dc.y * scale);
            out[N2] = make_float2(x.mid.x * scale, x.mid.y * scale);
            out[N2 / 2] = make_float2(x.q1.x * scale, x.q1.y * scale);
            out[N2 + N2 / 2] = make_float2(x.q3.x * scale, x.q3.y * scale);
        } else {
            const Quad x = quad_forward(A[pad0(k)], A[pad0(N2 - k)], Bf[pad0(k)], Bf[pad0(N2 - k)],
                                        __ldg(&tw[tw_index(NB2, k)]), __ldg(&tw[tw_index(F2, k)]));
            out[k] = make_float2(x.k.x * scale, x.k.y * scale);
            out[NB2 - k] = make_float2(x.nk.x * scale, x.nk.y * scale);
            out[N2 - k] = make_float2(x.mk.x * scale, x.mk.y * scale);
            out[N2 + k] = make_float2(x.pk.x * scale, x.pk.y * scale);
        }
    }
}

// What the spectral phase reads from global memory for slot k: the join and split
// twiddles and the four response bins X[k], X[8192-k], X[4096-k], X[4096+k] pair with
// (slot 0: the split twiddle of bin 2048 and bins 0/8192, 4096, 2048, 6144).
struct SpecOps {
    float2 w, u, h0, h1, h2, h3;
};
__device__ __forceinline__ SpecOps load_spec_ops(const float2 *__restrict__ H, const float2 *__restrict__ tw,
                                                 int k) {
    SpecOps o;
    const bool z = k == 0;
    o.w = __ldg(&tw[tw_index(NB2, k)]);
    o.u = __ldg(&tw[z ? tw_index(F2, N2 / 2) : tw_index(F2, k)]);
    o.h0 = __ldg(&H[k]);
    o.h1 = __ldg(&H[z ? N2 : NB2 - k]);
    o.h2 = __ldg(&H[z ? N2 / 2 : N2 - k]);
    o.h3 = __ldg(&H[z ? N2 + N2 / 2 : N2 + k]);
    return o;
}

// PARK: rows may have several noise sources (the context allows three or more
// sources); without it the kernel carries none of the parking code.
template <bool PARK>
__global__ void __launch_bounds__(CT, CONV_MINB)
convolve_fused2_kernel(const float *__restrict__ speech, int64_t stride,
                       const int *__restrict__ lengths, const float *__restrict__ bank,
                       int64_t bank_len, const AugUttParams *__restrict__ table, int S_max,
                       const float2 *__restrict__ hspec, const float2 *__restrict__ tw,
                       float *__restrict__ ys, float *__restrict__ vv, int64_t ws_stride,
                       double *__restrict__ energy, int *status, int n_cap,
                       const int *__restrict__ leff, const int *__restrict__ leff_all, int64_t hs_stride,
                       int mixed,
                       float2 *__restrict__ park, int *park_flags, int n_sm) {
    extern __shared__ __align__(16) float2 sm[];
    float2 *A = sm, *Bf = sm + SM_POINTS;
    __shared__ float red[CT / 32];
    __shared__ int park_slot_s;
    const int b = blockIdx.x, utt = blockIdx.y, t = threadIdx.x;
    const int N = min(max(lengths[utt], 0), n_cap);
    // every block yields the F2 - (taps - 1) outputs that see no wrap-around, cut to a multiple
    // of 4, where taps counts up to the last non-zero tap of this utterance's responses
    if (mixed && !takes_fused_route(*leff_all)) return;
    const int taps_used = leff[utt];
    const int ob = (F2 - min(max(taps_used, 1), BLK2) + 1) & ~3;
    if ((int64_t)b * ob >= N) return;
    const AugUttParams &row = table[utt];
    int n_src = row.n_src;
    if (n_src < 1 || n_src > S_max) n_src = 0;   // rejected row: silence (reported by step 1)
    const int m0 = (F2 - ob) / 4;            // first point of A and B that belongs to a block

    int last_noise = 0, n_noise = 0;
    for (int s = 1; s < n_src; ++s) {
        const float *x;
        int nlen;
        if (source_of(row, s, nullptr, bank, bank_len, x, nlen)) {
            last_noise = s;
            ++n_noise;
        } else if (t == 0 && b == 0 && atomicCAS(&status[0], -1, utt) == -1) {
            status[1] = aug::R_NOISE;
        }
    }
    // Several noise sources are summed in the frequency domain: the products of all
    // but the last are parked in a 64 KB global slot (one per resident CTA of an SM,
    // taken with a compare-and-swap; it stays in L2) and added to the last one's
    // before the single inverse transform.  A CTA that finds no free slot -- more
    // CTAs on the SM than slots -- sums in the time domain instead: v is read back
    // and added to for every source after the first, one inverse transform each.
    int park_slot = -1;
    if (PARK && n_noise > 1 && park != nullptr) {
        if (t == 0) {
            unsigned smid;
            asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
            int got = -1;
            if ((int)smid < n_sm) {
                for (int i = 0; i < CONV_MINB && got < 0; ++i)
                    if (atomicCAS(&park_flags[smid * CONV_MINB + i], 0, 1) == 0) got = smid * CONV_MINB + i;
            }
            park_slot_s = got;
        }
        __syncthreads();
        park_slot = park_slot_s;
    }
    float2 *slot = park_slot >= 0 ? park + (int64_t)park_slot * (4 * NQ2 * CT) : nullptr;
    const int n_left = min(N - b * ob, ob);
    bool v_written = false, v_parked = false;
    for (int s = 0; s < n_src; ++s) {
        const float *x;
        int nlen;
        if (!source_of(row, s, speech + (int64_t)utt * stride, bank, bank_len, x, nlen)) continue;
        {
            float2 va[1][E], vb[1][E];
            load_segment4(va, vb, x, s != 0, nlen, (b + 1) * ob - F2, N, t, bank + bank_len);
            fft2x4096_from_regs(va, vb, A, Bf, t, tw);
        }
        const float2 *H = hspec + ((int64_t)utt * S_max + s) * hs_stride;
        // the first slot's operands are requested before the barrier that completes the transform
        SpecOps nxt = load_spec_ops(H, tw, t);
        __syncthreads();
        // what happens to this source's products: inverse-transformed right away (0),
        // parked for a later noise source (1: first one, 2: added to what is parked),
        // or joined by the parked sum before the inverse (3)
        int mode = 0;
        if (PARK && s != 0 && slot != nullptr) mode = s == last_noise ? 3 : (v_parked ? 2 : 1);
#pragma unroll 2
        for (int q = 0; q < NQ2; ++q) {
            const int k = t + CT * q;
            const SpecOps c = nxt;
            if (q + 1 < NQ2) nxt = load_spec_ops(H, tw, k + CT);     // next slot's operands while this one is worked on
            float2 *pk = slot + (4 * q) * CT + t;      // this thread's four parked products, CT apart
            if (k == 0) {
                const float2 uh = c.u;
                Edge x4 = edge_forward(A[pad0(0)], Bf[pad0(0)], A[pad0(N2 / 2)], Bf[pad0(N2 / 2)], uh);
                x4.dc = make_float2(x4.dc.x * c.h0.x, x4.dc.y * c.h0.y);
                x4.mid = cmul(x4.mid, c.h1);
                x4.q1 = cmul(x4.q1, c.h2);
                x4.q3 = cmul(x4.q3, c.h3);
                if (PARK && mode >= 2) {
                    x4.dc = cadd(x4.dc, pk[0]);
                    x4.mid = cadd(x4.mid, pk[CT]);
                    x4.q1 = cadd(x4.q1, pk[2 * CT]);
                    x4.q3 = cadd(x4.q3, pk[3 * CT]);
                }
                if (PARK && (mode == 1 || mode == 2)) {
                    pk[0] = x4.dc;
                    pk[CT] = x4.mid;
                    pk[2 * CT] = x4.q1;
                    pk[3 * CT] = x4.q3;
                } else {
                    edge_inverse(x4, uh, A[pad0(0)], Bf[pad0(0)], A[pad0(N2 / 2)], Bf[pad0(N2 / 2)]);
                }
            } else {
                const float2 w = c.w, u = c.u;
                Quad x4 = quad_forward(A[pad0(k)], A[pad0(N2 - k)], Bf[pad0(k)], Bf[pad0(N2 - k)], w, u);
                x4.k = cmul(x4.k, c.h0);
                x4.nk = cmul(x4.nk, c.h1);
                x4.mk = cmul(x4.mk, c.h2);
                x4.pk = cmul(x4.pk, c.h3);
                if (PARK && mode >= 2) {
                    x4.k = cadd(x4.k, pk[0]);
                    x4.nk = cadd(x4.nk, pk[CT]);
                    x4.mk = cadd(x4.mk, pk[2 * CT]);
                    x4.pk = cadd(x4.pk, pk[3 * CT]);
                }
                if (PARK && (mode == 1 || mode == 2)) {
                    pk[0] = x4.k;
                    pk[CT] = x4.nk;
                    pk[2 * CT] = x4.mk;
                    pk[3 * CT] = x4.pk;
                } else {
                    quad_inverse(x4, w, u, A[pad0(k)], A[pad0(N2 - k)], Bf[pad0(k)], Bf[pad0(N2 - k)]);
                }
            }
        }
        if (PARK && (mode == 1 || mode == 2)) {
            // every thread reads back only what it parked itself: no fence is needed
            v_parked = true;
            __syncthreads();   // the buffers are refilled by the next source
            continue;
        }
        __syncthreads();
        fft2x4096_in_place(A, Bf, t, tw);
        __syncthreads();

        // The last `ob` outputs of the segment are this block: samples 4m, 4m+1 of the
        // segment are point m of A, samples 4m+2, 4m+3 point m of B.
        const bool is_speech = s == 0;
        const bool add = !is_speech && v_written;
        const bool want_energy = is_speech || s == last_noise;
        float *dst = (is_speech ? ys : vv) + (int64_t)utt * ws_stride + (int64_t)b * ob;
        float e2sum = 0.f;
        if (n_left >= ob) {
            // a whole block of outputs (the same for the CTA): no test per group
#pragma unroll 4
            for (int j = t; m0 + j < N2; j += CT) {
                const float2 za = A[pad0(m0 + j)], zb = Bf[pad0(m0 + j)];
                float4 y = make_float4(za.y, za.x, zb.y, zb.x);
                float4 *p = reinterpret_cast<float4 *>(dst + 4 * j);
                if (add) {
                    const float4 o = *p;
                    y = make_float4(y.x + o.x, y.y + o.y, y.z + o.z, y.w + o.w);
                }
                *p = y;
                e2sum += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
            }
        } else
#pragma unroll 4
        for (int j = t; m0 + j < N2; j += CT) {
            const float2 za = A[pad0(m0 + j)], zb = Bf[pad0(m0 + j)];
            float4 y = make_float4(za.y, za.x, zb.y, zb.x);
            const int i = 4 * j;
            if (i + 3 < n_left) {
                float4 *p = reinterpret_cast<float4 *>(dst + i);
                if (add) {
                    const float4 o = *p;
                    y = make_float4(y.x + o.x, y.y + o.y, y.z + o.z, y.w + o.w);
                }
                *p = y;
                e2sum += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
            } else {
                const float yy[3] = {y.x, y.y, y.z};
                for (int c = 0; c < 3 && i + c < n_left; ++c) {
                    const float val = add ? yy[c] + dst[i + c] : yy[c];
                    dst[i + c] = val;
                    e2sum += val * val;
                }
            }
        }
        if (want_energy) {
            const float tot = block_sum(e2sum, red, t);
            if (t == 0) atomicAdd(&energy[2 * utt + (is_speech ? 0 : 1)], (double)tot);
        }
        if (!is_speech) v_written = true;
        __syncthreads();   // the buffers are refilled by the next source
    }
    if (n_src == 0) {
        // rejected row: y_s is silence too
        float *dst = ys + (int64_t)utt * ws_stride + (int64_t)b * ob;
        for (int i = t; i < n_left; i += CT) dst[i] = 0.f;
    }
    if (!v_written) {
        // no (usable) noise: v is defined as silence
        float *dst = vv + (int64_t)utt * ws_stride + (int64_t)b * ob;
        for (int i = t; i < n_left; i += CT) dst[i] = 0.f;
    }
    if (PARK && park_slot >= 0) {
        __syncthreads();                                  // all reads of the slot are done
        if (t == 0) atomicExch(&park_flags[park_slot], 0);
    }
}

constexpr size_t FFT_SMEM = sizeof(float2) * SM_POINTS;
constexpr size_t FFT2_SMEM = 2 * FFT_SMEM;

}  // namespace

static bool stored_route(const AugCtx *ctx) { return ctx->route == aug::ROUTE_STORED; }
// response spectra of one (utterance, source): complex numbers between consecutive ones
static int64_t hspec_stride(const AugCtx *ctx) { return stored_route(ctx) ? (int64_t)ctx->n_part * N2 : NB2; }

int launch_rir_spectra(AugCtx *ctx, const float *rir, const AugUttParams *table, int B,
                       cudaStream_t st) {
    const AugConfig &c = ctx->cfg;
    const int mixed = stored_route(ctx) ? 1 : 0;
    // long-response context: the last batch size seen decides whether the fused kernels are launched at all
    ctx->stored_only = mixed && ctx->leff_seen && *ctx->leff_seen > BLK2;
    int *leff_all = ctx->leff + ctx->cfg.max_batch;
    AUG_CUDA_OK(cudaMemsetAsync(ctx->leff, 0, sizeof(int) * (size_t)B, st));
    AUG_CUDA_OK(cudaMemsetAsync(leff_all, 0, sizeof(int), st));
    dim3 grid2(c.max_sources, B);
    if (mixed) {
        rir_length_kernel<<<grid2, CT, 0, st>>>(rir, table, c.max_sources, c.rir_taps, ctx->leff, leff_all);
        AUG_CUDA_OK(cudaGetLastError());
        ctx->launches++;
    }
    if (!ctx->stored_only) {
        if (smem_opt_in<rir_spectra2_kernel>(ctx->device) != AUG_OK) return AUG_ECUDA;
        rir_spectra2_kernel<<<grid2, CT, FFT2_SMEM, st>>>(rir, table, c.max_sources, c.rir_taps, ctx->tw,
                                                          ctx->hspec, hspec_stride(ctx), ctx->leff, leff_all,
                                                          mixed);
        AUG_CUDA_OK(cudaGetLastError());
        ctx->launches++;
    }
    if (mixed) {
        dim3 grid(ctx->n_part, c.max_sources, B);
        rir_spectra_kernel<<<grid, CT, FFT_SMEM, st>>>(rir, table, c.max_sources, c.rir_taps,
                                                       ctx->n_part, ctx->tw, ctx->hspec, leff_all,
                                                       ctx->stored_only);
        AUG_CUDA_OK(cudaGetLastError());
        ctx->launches++;
    }
    return AUG_OK;
}

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
        ctx->nblk_cap, ctx->status, max_len, ctx->leff + c.max_batch, ctx->stored_only);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

int launch_convolve_finish(AugCtx *ctx, const float *speech, int64_t stride, const int *lengths,
                           const float *bank, int64_t bank_len, const AugUttParams *table, int B,
                           int max_len) {
    const AugConfig &c = ctx->cfg;
    if (max_len <= 0) return AUG_OK;
    const int mixed = stored_route(ctx) ? 1 : 0;
    const int *leff_all = ctx->leff + c.max_batch;
    if (!ctx->stored_only) {
        // fused route: the grid covers the shortest block an utterance on it can have (a response
        // that fills min(rir_taps, 8192) taps)
        const int ob_min = (F2 - min(c.rir_taps, BLK2) + 1) & ~3;
        const int nblk2 = (max_len + ob_min - 1) / ob_min;
        dim3 grid2(nblk2, B);
        auto kern = ctx->park ? convolve_fused2_kernel<true> : convolve_fused2_kernel<false>;
        if ((ctx->park ? smem_opt_in<convolve_fused2_kernel<true>>(ctx->device)
                       : smem_opt_in<convolve_fused2_kernel<false>>(ctx->device)) != AUG_OK)
            return AUG_ECUDA;
        kern<<<grid2, CT, FFT2_SMEM, ctx->stream>>>(
            speech, stride, lengths, bank, bank_len, table, c.max_sources, ctx->hspec, ctx->tw,
            ctx->ys, ctx->vv, ctx->ws_stride, ctx->energy, ctx->status, max_len, ctx->leff, leff_all,
            hspec_stride(ctx), mixed, ctx->park, ctx->park_flags, ctx->n_sm);
        AUG_CUDA_OK(cudaGetLastError());
        ctx->launches++;
    }
    if (mixed) {
        const int nblk = (max_len + BLK - 1) / BLK;
        dim3 grid(nblk, B);
        spectral_convolve_kernel<<<grid, CT, FFT_SMEM, ctx->stream>>>(
            lengths, bank, bank_len, table, c.max_sources, ctx->n_part, ctx->hspec, ctx->xspec,
            ctx->nblk_cap, ctx->tw, ctx->ys, ctx->vv, ctx->ws_stride, ctx->energy, max_len, ctx->leff, leff_all,
            ctx->stored_only);
        AUG_CUDA_OK(cudaGetLastError());
        ctx->launches++;
        // for the next call's choice (not waited for)
        if (ctx->leff_seen)
            AUG_CUDA_OK(cudaMemcpyAsync(ctx->leff_seen, leff_all, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    }
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
