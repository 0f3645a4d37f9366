// Waveform-domain VTLP: the warp of Eq. 1 applied to the speech itself, with
// resynthesis, before the simulator (Section 2.3; 50 ms window of Section 4).
//
// The paper prints only the frequency map.  The reading built here: frames of
// `win` samples every win/4, periodic Hann, the utterance zero-padded by
// win - win/4 samples in front; 1024-point DFT; the spectrum at bin k becomes the
// old spectrum at the frequency that Eq. 1 moves to bin k (the all-pass with the
// opposite coefficient), by linear interpolation between the two nearest bins;
// inverse DFT, first `win` samples, Hann again, overlap-add, division by the sum
// of the squared windows.
//
// Two frames ride through the transforms as the real and imaginary part of one
// complex signal: interpolation is linear, so it acts on the packed spectrum Z
// directly (bin k from Z around k0, bin K-k from Z around K-k0), and the inverse of
// the packed spectrum returns the two frames in its real and imaginary part.
// A CTA owns the output samples of HB hops and computes the HB + 3 frames that
// cover them, so nothing is added across CTAs: four 64-thread groups transform a
// frame pair each, then every thread adds what the round's frames contribute to the
// output samples it owns (in registers), and so on for the next round.
#include "common.cuh"
#include "fft.cuh"

namespace {

using namespace augfft;
constexpr int K = 1024;
constexpr int E = 16;                 // points per thread
constexpr int GROUP = K / E;          // 64 threads per transform
constexpr int NGROUP = 4;
constexpr int RS_THREADS = GROUP * NGROUP;
#ifndef RS_HB
#define RS_HB 13
#endif
constexpr int HB = RS_HB;             // hops of output per CTA: 13 + 3 frames = 8 pairs, two full rounds of the four groups
constexpr int NF = HB + 3;            // frames that cover them
constexpr int XB = padded_points(K);

__host__ __device__ constexpr size_t resynth_smem(int win) {
    const int hop = win / 4;
    return sizeof(float2) * 2 * NGROUP * XB + sizeof(float) * (size_t)((NF - 1) * hop + win) +
           sizeof(float) * win + sizeof(float) * (K / 2 + 1) + sizeof(int) * (K / 2 + 1);
}

__device__ __forceinline__ void fft1024_from_regs(float2 (*v)[E], float2 *s, int tg, const float2 *__restrict__ tw,
                                                  GroupSync gsync) {
    pass_from_regs<K, E, E, 1>(v, s, tg, tw);
    gsync();
    pass<K, E, 8, 16, 1>(s, tg, tw, gsync);
    pass<K, E, 8, 128, 16>(s, tg, tw, gsync);
}
__device__ __forceinline__ void fft1024_in_place(float2 *s, int tg, const float2 *__restrict__ tw, GroupSync gsync) {
    pass<K, E, E, 1, 0>(s, tg, tw, gsync);
    pass<K, E, 8, 16, 1>(s, tg, tw, gsync);
    pass<K, E, 8, 128, 16>(s, tg, tw, gsync);
}

// Source position of every bin of an utterance: the frequency that Eq. 1 moves to bin k, in
// bins, as lower bin and fraction (fp64: a position error of 6e-5 bins, one fp32 ulp at bin 512,
// would already cost half of the waveform tolerance).
__global__ void __launch_bounds__(256)
vtlp_positions_kernel(const AugUttParams *__restrict__ table, int *__restrict__ k0_tab,
                      float *__restrict__ fr_tab) {
    const int utt = blockIdx.x;
    const double a = 1.0 - (double)table[utt].alpha;
    const double PI = 3.14159265358979323846;
    for (int k = threadIdx.x; k <= K / 2; k += 256) {
        const double om = 2.0 * PI * k / K;
        double pos = (om - 2.0 * atan(a * sin(om) / (1.0 + a * cos(om)))) * K / (2.0 * PI);
        if (k == 0) pos = 0.0;
        if (k == K / 2) pos = (double)(K / 2);
        int k0 = (int)floor(pos);
        k0 = min(max(k0, 0), K / 2 - 1);
        k0_tab[(int64_t)utt * (K / 2 + 1) + k] = k0;
        fr_tab[(int64_t)utt * (K / 2 + 1) + k] = (float)(pos - (double)k0);
    }
}

__global__ void __launch_bounds__(RS_THREADS, 2)
vtlp_resynth_kernel(const float *__restrict__ speech, int64_t stride, const int *__restrict__ lengths,
                    const int *__restrict__ k0_tab, const float *__restrict__ fr_tab, int win,
                    const float2 *__restrict__ tw, float *__restrict__ out, int64_t out_stride, int n_cap) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int hop = win >> 2, front = win - hop;
    float2 *zbuf = reinterpret_cast<float2 *>(smem_raw);            // [NGROUP][XB] forward transforms
    float2 *wbuf = zbuf + NGROUP * XB;                              // [NGROUP][XB] warped spectra / inverse
    float *xin = reinterpret_cast<float *>(wbuf + NGROUP * XB);     // [(NF-1) hop + win] padded input stretch
    float *wn = xin + (NF - 1) * hop + win;                         // [win] Hann
    float *fr_s = wn + win;                                         // [K/2+1] interpolation fraction
    int *k0_s = reinterpret_cast<int *>(fr_s + K / 2 + 1);          // [K/2+1] lower source bin

    const int utt = blockIdx.y, tid = threadIdx.x, tg = tid & (GROUP - 1), grp = tid / GROUP;
    const int N = min(max(lengths[utt], 0), n_cap);
    if (N == 0) return;
    const int T = (N + front + hop - 1) / hop;       // frames = hops that cover the padded utterance
    const int t0 = blockIdx.x * HB;                  // first hop this CTA owns
    if (t0 >= T) return;
    const float *x = speech + (int64_t)utt * stride;
    float *y = out + (int64_t)utt * out_stride;

    for (int k = tid; k <= K / 2; k += RS_THREADS) {
        k0_s[k] = k0_tab[(int64_t)utt * (K / 2 + 1) + k];
        fr_s[k] = fr_tab[(int64_t)utt * (K / 2 + 1) + k];
    }
    for (int n = tid; n < win; n += RS_THREADS) wn[n] = 0.5f - 0.5f * cospif(2.f * (float)n / (float)win);
    // input stretch of frames t0-3 .. t0+HB-1 in padded coordinates
    const int c0 = (t0 - 3) * hop;
    for (int i = tid; i < (NF - 1) * hop + win; i += RS_THREADS) {
        const int idx = c0 + i - front;
        xin[i] = (idx >= 0 && idx < N) ? x[idx] : 0.f;
    }
    __syncthreads();

    float2 *Z = zbuf + grp * XB, *W = wbuf + grp * XB;
    const GroupSync gsync{grp + 1, GROUP};
    constexpr int NPAIR = (NF + 1) / 2;
    constexpr int OWN = (HB * 256 + RS_THREADS - 1) / RS_THREADS;   // owned samples per thread (hop <= 256)
    float acc[OWN];
#pragma unroll
    for (int u = 0; u < OWN; ++u) acc[u] = 0.f;
    const float inv_k = 1.f / (float)K, inv_hop = 1.f / (float)hop;

    for (int round = 0; round * NGROUP < NPAIR; ++round) {
        const int pr = round * NGROUP + grp;
        const int fa = 2 * pr, fb = fa + 1;                       // frame slots; frame number = t0 - 3 + slot
        const bool have_a = fa < NF && t0 - 3 + fa >= 0 && t0 - 3 + fa < T;
        const bool have_b = fb < NF && t0 - 3 + fb >= 0 && t0 - 3 + fb < T;
        if (have_a || have_b) {                                   // (uniform over the group)
            {
                float2 v[1][E];
#pragma unroll
                for (int r = 0; r < E; ++r) {
                    const int n = tg + GROUP * r;
                    float a = 0.f, b = 0.f;
                    if (n < win) {
                        const float w = wn[n];
                        if (have_a) a = w * xin[fa * hop + n];
                        if (have_b) b = w * xin[fb * hop + n];
                    }
                    v[0][r] = make_float2(a, b);
                }
                fft1024_from_regs(v, Z, tg, tw, gsync);
            }
            // warped packed spectrum, real and imaginary parts swapped for the inverse
            for (int k = tg; k <= K / 2; k += GROUP) {
                const int k0 = k0_s[k];
                const float fr = fr_s[k], om = 1.f - fr;
                const float2 z0 = Z[pad0(k0)], z1 = Z[pad0(k0 + 1)];
                W[pad0(k)] = make_float2(fmaf(fr, z1.y, om * z0.y), fmaf(fr, z1.x, om * z0.x));
                if (k > 0 && k < K / 2) {
                    const float2 m0 = Z[pad0((K - k0) & (K - 1))], m1 = Z[pad0(K - k0 - 1)];
                    W[pad0(K - k)] = make_float2(fmaf(fr, m1.y, om * m0.y), fmaf(fr, m1.x, om * m0.x));
                }
            }
            gsync();
            fft1024_in_place(W, tg, tw, gsync);               // W[n] = (imaginary, real) of the inverse, times K
        }
        __syncthreads();
        // What this round's frames add to the owned samples.  Sample i of the CTA lies in hop
        // q = i / hop at offset r and is covered by the four frames in slots q .. q + 3, at
        // n = r + (3 - d) hop of slot q + d; this round holds slots 8 round .. 8 round + 7
        // (group g: slots 2 g and 2 g + 1, in the imaginary and real part of its buffer).
#pragma unroll
        for (int u = 0; u < OWN; ++u) {
            const int i = tid + u * RS_THREADS;
            if (i < HB * hop) {
                const int q = (int)(((float)i + 0.5f) * inv_hop);      // exact: i + 1/2 is never a multiple of hop
                const int r = i - q * hop;
                float sum = 0.f;
#pragma unroll
                for (int d = 0; d < 4; ++d) {
                    const int gl = q + d - 2 * NGROUP * round, t = t0 - 3 + q + d;
                    if ((unsigned)gl < (unsigned)(2 * NGROUP) && t >= 0 && t < T) {
                        const int n = r + (3 - d) * hop;
                        const float *Wf = reinterpret_cast<const float *>(wbuf + (gl >> 1) * XB);
                        sum = fmaf(wn[n], Wf[2 * n + 1 - (gl & 1)], sum);
                    }
                }
                acc[u] = fmaf(sum, inv_k, acc[u]);
            }
        }
        __syncthreads();      // the buffers are refilled in the next round
    }

    // owned samples: sample c is covered by frames c/hop - 3 .. c/hop; divide by their squared windows
#pragma unroll
    for (int u = 0; u < OWN; ++u) {
        const int i = tid + u * RS_THREADS;
        const int c = t0 * hop + i;
        const int idx = c - front;
        if (i >= HB * hop || idx < 0 || idx >= N) continue;
        const int hb = t0 + i / hop;
        float norm = 0.f;
#pragma unroll
        for (int d = 0; d < 4; ++d) {
            const int t = hb - d;
            if (t >= 0 && t < T) {
                const float w = wn[c - t * hop];
                norm = fmaf(w, w, norm);
            }
        }
        y[idx] = acc[u] / norm;
    }
}

}  // namespace

int launch_vtlp_resynth(AugCtx *ctx, const float *speech, int64_t stride, const int *lengths,
                        const AugUttParams *table, int B, int max_len, float *out, int64_t out_stride) {
    const int win = ctx->cfg.vtlp_win;
    if (win <= 0 || max_len <= 0) return AUG_OK;
    const int hop = win / 4, front = win - hop;
    const int T_cap = (max_len + front + hop - 1) / hop;
    const size_t smem = resynth_smem(win);
    if (smem_opt_in<vtlp_resynth_kernel>(ctx->device) != AUG_OK) return AUG_ECUDA;
    int *k0_tab = reinterpret_cast<int *>(ctx->vtlp_tab);
    float *fr_tab = reinterpret_cast<float *>(k0_tab + (size_t)ctx->cfg.max_batch * (K / 2 + 1));
    vtlp_positions_kernel<<<B, 256, 0, ctx->stream>>>(table, k0_tab, fr_tab);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    dim3 grid((T_cap + HB - 1) / HB, B);
    vtlp_resynth_kernel<<<grid, RS_THREADS, smem, ctx->stream>>>(speech, stride, lengths, k0_tab, fr_tab, win,
                                                                ctx->tw, out, out_stride, max_len);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}
