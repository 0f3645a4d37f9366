// Steps 3 and 4: framing, Hann window, power spectrum, VTLP-warped mel
// filterbank and compression -- separately (stft_power / logmel kernels) and
// fused with the SNR mix (fused kernel: y_s + g v -> features, the power
// spectrum never leaves shared memory).
//
// A CTA owns a tile of FT consecutive frames of one utterance.  It stages the
// contiguous stretch of samples those frames cover in shared memory once, then
// groups of 64 threads transform two frames at a time as the real and imaginary
// part of one complex K-point FFT and separate the two spectra afterwards.
// The filterbank is applied as a gather: band m sums the bins of edge interval m
// with their rising weights and those of interval m+1 with their falling
// weights; the intervals are contiguous bin ranges because the warp of Eq. 1 is
// monotone.  The fused kernel walks every interval once and keeps both sums.
#include "common.cuh"
#include "fft.cuh"

namespace {

using namespace augfft;
constexpr int FEAT_THREADS = 256;
constexpr int GROUP = 64;                         // threads per FFT
constexpr int NGROUP = FEAT_THREADS / GROUP;

__host__ __device__ __forceinline__ int frame_count(int n, int win, int hop) {
    return n >= win ? 1 + (n - win) / hop : 0;
}

// ---------------------------------------------------------------- filterbank tables
// One CTA per utterance: per DFT bin the edge interval and weights at the warped
// frequency (fp64: a bin that barely enters a band must not lose its weight to
// rounding), then the first bin of every interval.
__global__ void __launch_bounds__(256)
mel_tables_kernel(const AugUttParams *__restrict__ table, int K, int M, double fs, double f_lo,
                  double f_hi, aug::MelBin *__restrict__ melw, int *__restrict__ melstart, int unwarped) {
    __shared__ int seg_s[513];
    const int utt = blockIdx.x, nb = K / 2 + 1;
    // (unwarped: the warp was already applied to the waveform)
    const double a = unwarped ? 0.0 : 1.0 - (double)table[utt].alpha;
    const double PI = 3.14159265358979323846;
    const double e0 = 2595.0 * log10(1.0 + f_lo / 700.0);
    const double e1 = 2595.0 * log10(1.0 + f_hi / 700.0);
    const double delta = (e1 - e0) / (M + 1);
    for (int k = threadIdx.x; k < nb; k += blockDim.x) {
        const double om = 2.0 * PI * k / K;
        const double omw = om + 2.0 * atan(a * sin(om) / (1.0 - a * cos(om)));   // Eq. 1
        const double fw = omw * fs / (2.0 * PI);
        const double mu = 2595.0 * log10(1.0 + fw / 700.0);
        const double u = (mu - e0) / delta;
        int seg;
        aug::MelBin w;
        if (!(u >= 0.0)) {
            seg = -1;
            w.up = w.down = 0.f;
        } else if (u >= (double)(M + 1)) {
            seg = M + 1;
            w.up = w.down = 0.f;
        } else {
            const double fl = floor(u);
            seg = (int)fl;
            w.up = (float)(u - fl);
            w.down = (float)(1.0 - (u - fl));
        }
        seg_s[k] = seg;
        melw[(int64_t)utt * nb + k] = w;
    }
    int *st = melstart + (int64_t)utt * (M + 2);
    for (int m = threadIdx.x; m < M + 2; m += blockDim.x) st[m] = nb;
    __syncthreads();
    for (int k = threadIdx.x; k < nb; k += blockDim.x) {
        const int prev = k ? seg_s[k - 1] : -1;
        const int cur = seg_s[k];
        for (int m = prev + 1; m <= cur && m < M + 2; ++m) st[m] = k;   // first bin with seg >= m
    }
}

// Filterbank energy of band m for one frame's power spectrum `p`.
__device__ __forceinline__ float band_energy(const float *p, const aug::MelBin *w, const int *st,
                                             int m) {
    float e = 0.f;
    const int k0 = st[m], k1 = st[m + 1], k2 = st[m + 2];
    for (int k = k0; k < k1; ++k) e = fmaf(w[k].up, p[k], e);
    for (int k = k1; k < k2; ++k) e = fmaf(w[k].down, p[k], e);
    return e;
}

__device__ __forceinline__ float compress(float e, float floor_v, int mode) {
    e = fmaxf(e, floor_v);
    const float l = logf(e);
    return mode == AUG_COMPRESS_LOG ? l : expf(l * (1.f / 15.f));
}

// ---------------------------------------------------------------- tile transform
// Power spectra of `nf` frames starting `hop` apart in `chunk` (shared memory)
// into ptile[f][k], k <= K/2 (row stride K/2+1).
// Window values of the E points a thread holds (n = tg + GROUP r), zero beyond the window.
template <int E>
__device__ __forceinline__ void window_values(float *wv, int win) {
    const int tg = threadIdx.x & (GROUP - 1);
#pragma unroll
    for (int r = 0; r < E; ++r) {
        const int n = tg + GROUP * r;
        wv[r] = n < win ? 0.5f - 0.5f * cospif(2.f * (float)n / (float)win) : 0.f;
    }
}

template <int K, int E>
__device__ __forceinline__ void tile_power(const float *chunk, int nf, int win, int hop,
                                           const float *wv, float2 *fbuf, float *ptile,
                                           const float2 *__restrict__ tw) {
    static_assert(K / E == GROUP, "one FFT per 64-thread group");
    const int tid = threadIdx.x, tg = tid & (GROUP - 1), grp = tid / GROUP;
    float2 *s = fbuf + grp * padded_points(K);
    constexpr int NBP = K / 2 + 1;
    const GroupSync gsync{grp + 1, GROUP};
    const int npair = (nf + 1) / 2;
    const int iters = (npair + NGROUP - 1) / NGROUP;
    for (int it = 0; it < iters; ++it) {
        const int pr = it * NGROUP + grp;
        const int f0 = 2 * pr;
        const bool have0 = f0 < nf, have1 = f0 + 1 < nf;
        float2 v[1][E];
#pragma unroll
        for (int r = 0; r < E; ++r) {
            const int n = tg + GROUP * r;
            float a = 0.f, b = 0.f;
            if (n < win) {
                if (have0) a = wv[r] * chunk[f0 * hop + n];
                if (have1) b = wv[r] * chunk[(f0 + 1) * hop + n];
            }
            v[0][r] = make_float2(a, b);
        }
        // each 64-thread group runs its transforms on its own hardware barrier
        if constexpr (K == 512) {
            pass_from_regs<K, E, 8, 1>(v, s, tg, tw);
            gsync();
            pass<K, E, 8, 8, 1>(s, tg, tw, gsync);
            pass<K, E, 8, 64, 8>(s, tg, tw, gsync);
        } else {
            pass_from_regs<K, E, E, 1>(v, s, tg, tw);
            gsync();
            pass<K, E, 8, 16, 1>(s, tg, tw, gsync);
            pass<K, E, 8, 128, 16>(s, tg, tw, gsync);
        }
        if (have0) {
            float *p0 = ptile + f0 * NBP, *p1 = p0 + NBP;
            for (int k = tg; k <= K / 2; k += GROUP) {
                const float2 z = s[pad0(k)], q = s[pad0((K - k) & (K - 1))];
                const float ar = z.x + q.x, ai = z.y - q.y;
                const float br = z.y + q.y, bi = z.x - q.x;
                p0[k] = 0.25f * (ar * ar + ai * ai);
                if (have1) p1[k] = 0.25f * (br * br + bi * bi);
            }
        }
        gsync();   // the group's buffer is rewritten by its next pair
    }
    __syncthreads();   // all power spectra of the tile are in place
}

#ifndef FEAT_FT_512
#define FEAT_FT_512 32      // frames per CTA tile, 512-point transform
#endif
#ifndef FEAT_FT_1024
#define FEAT_FT_1024 8      // frames per CTA tile, 1024-point transform (64 KB of shared memory: 3 CTAs/SM)
#endif
#ifndef FEAT_TILES_1024
#define FEAT_TILES_1024 8   // consecutive tiles one CTA works through, 1024-point transform
#endif
#ifndef FEAT_TILES
#define FEAT_TILES 4        // consecutive tiles one CTA works through
#endif
template <int K>
struct Plan;
template <>
struct Plan<512> {
    static constexpr int E = 8, FT = FEAT_FT_512, TILES = FEAT_TILES;
};
template <>
struct Plan<1024> {
    static constexpr int E = 16, FT = FEAT_FT_1024, TILES = FEAT_TILES_1024;
};

// Floats of the region that first holds the transform buffers of the four groups and
// then, once a tile's transforms are done, the two interval sums [FT][M+1] of the filterbank.
template <int K>
__host__ __device__ constexpr int fbuf_floats(int FT, int M) {
    const int a = 2 * NGROUP * padded_points(K), b = 2 * FT * (M + 1);
    return ((a > b ? a : b) + 3) & ~3;
}

#ifndef FEAT_MINB
#define FEAT_MINB 3           // CTAs per SM the register budget is set for
#endif
// MODE 0: wave -> power (global).  MODE 1: y_s + g v -> features.
// TILES: consecutive tiles one CTA works through.
template <int K, int MODE, int TILES>
__global__ void __launch_bounds__(FEAT_THREADS, FEAT_MINB)
frames_kernel(const float *__restrict__ in_a, const float *__restrict__ in_b, int64_t in_stride,
              const float *__restrict__ gain, const AugUttParams *__restrict__ table,
              const int *__restrict__ lengths, int win, int hop, int M, int T_max,
              const aug::MelBin *__restrict__ melw, const int *__restrict__ melstart,
              const float2 *__restrict__ tw, float floor_v, float pad_v, int comp,
              float *__restrict__ out, int *__restrict__ counts, int n_cap) {
    constexpr int E = Plan<K>::E, FT = Plan<K>::FT, NBP = K / 2 + 1;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float2 *fbuf = reinterpret_cast<float2 *>(smem_raw);            // [NGROUP][K + K/8]; later the interval sums
    float *ptile = reinterpret_cast<float *>(smem_raw) + fbuf_floats<K>(FT, M);    // [FT][NBP]
    float *chunk = ptile + FT * NBP;                                // [(FT-1) hop + win] (+pad)
    const int chunk_cap = ((FT - 1) * hop + win + 3) & ~3;
    aug::MelBin *mw = reinterpret_cast<aug::MelBin *>(chunk + chunk_cap);   // [NBP]
    int *mst = reinterpret_cast<int *>(mw + NBP + 1);                       // [M+2]

    const int utt = blockIdx.y, tid = threadIdx.x;
    const int run0 = blockIdx.x * (FT * TILES);    // first frame of this CTA's run of tiles
    const int N = min(max(lengths[utt], 0), n_cap);
    const int T = min(frame_count(N, win, hop), T_max);
    if (blockIdx.x == 0 && tid == 0) counts[utt] = T;
    const int rows = min(FT * TILES, T_max - run0);     // rows of the output this run owns
    if (rows <= 0) return;
    const int nfr = max(0, min(FT * TILES, T - run0));  // of which real frames
    const int out_w = MODE == 0 ? NBP : M;
    float *orun = out + ((int64_t)utt * T_max + run0) * out_w;
    const float fill = MODE == 0 ? 0.f : pad_v;
    for (int i = nfr * out_w + tid; i < rows * out_w; i += FEAT_THREADS) orun[i] = fill;
    if (nfr == 0) return;

    const float g = MODE == 1 ? gain[utt] : 0.f;
    const float *ra = in_a + (int64_t)utt * in_stride;
    const float *rb = MODE == 1 ? in_b + (int64_t)utt * in_stride : nullptr;
    const bool vec = (hop & 3) == 0 && (in_stride & 3) == 0;
    if (MODE == 1) {
        for (int k = tid; k < NBP; k += FEAT_THREADS) mw[k] = melw[(int64_t)utt * NBP + k];
        for (int m = tid; m < M + 2; m += FEAT_THREADS) mst[m] = melstart[(int64_t)utt * (M + 2) + m];
    }
    float wv[E];
    window_values<E>(wv, win);
    const int out_f0 = tid / M, out_m0 = tid - out_f0 * M;                   // first output element of this thread
    const int step_f = FEAT_THREADS / M, step_m = FEAT_THREADS - step_f * M;  // and the stride to its next one

    for (int tile = 0; tile < TILES; ++tile) {
        const int t0 = run0 + tile * FT;
        const int nf = min(FT, T - t0);                 // frames of this tile
        if (nf <= 0) break;
        const int s0 = t0 * hop;
        const int ns = (nf - 1) * hop + win;            // samples they cover (all below N)
        const float *pa = ra + s0;
        const float *pb = MODE == 1 ? rb + s0 : nullptr;

        // Stage the samples of these frames.  All loads of a batch are issued before
        // the first is used: a tile costs one memory round trip, not one per 1024
        // samples.  The stretch of the next tile is pulled into L2 meanwhile.
        if (vec) {
            constexpr int SB = 6;                       // 128-bit loads per thread, array and batch
            for (int i0 = tid * 4; i0 < ns; i0 += SB * FEAT_THREADS * 4) {
                float4 xa[SB], xb[SB];
#pragma unroll
                for (int u = 0; u < SB; ++u) {
                    const int i = i0 + u * FEAT_THREADS * 4;
                    xa[u] = xb[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    // rows are allocated up to a multiple of 4 floats: whole groups can be read
                    if (i < ns) {
                        xa[u] = __ldg(reinterpret_cast<const float4 *>(pa + i));
                        if (MODE == 1 && g != 0.f) xb[u] = __ldg(reinterpret_cast<const float4 *>(pb + i));
                    }
                }
                if (i0 == tid * 4 && tile + 1 < TILES && t0 + FT < T) {
                    // next tile: FT hop samples further on, 128 bytes per prefetch
                    const int nxt = s0 + FT * hop + tid * 32;
                    if (nxt < N) {
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(ra + nxt));
                        if (MODE == 1 && g != 0.f) asm volatile("prefetch.global.L2 [%0];" ::"l"(rb + nxt));
                    }
                }
#pragma unroll
                for (int u = 0; u < SB; ++u) {
                    const int i = i0 + u * FEAT_THREADS * 4;
                    if (i < ns) {
                        float4 x = xa[u];
                        const float4 y = xb[u];
                        if (MODE == 0 && s0 + i + 3 >= N) {      // caller's buffer: nothing beyond N is used
                            if (s0 + i + 1 >= N) x.y = 0.f;
                            if (s0 + i + 2 >= N) x.z = 0.f;
                            x.w = 0.f;
                        }
                        *reinterpret_cast<float4 *>(chunk + i) = make_float4(
                            fmaf(g, y.x, x.x), fmaf(g, y.y, x.y), fmaf(g, y.z, x.z), fmaf(g, y.w, x.w));
                    }
                }
            }
        } else {
            for (int i = tid; i < ns; i += FEAT_THREADS)
                chunk[i] = (MODE == 1 && g != 0.f) ? fmaf(g, pb[i], pa[i]) : pa[i];
        }
        __syncthreads();

        tile_power<K, E>(chunk, nf, win, hop, wv, fbuf, ptile, tw);

        float *orow = orun + (int64_t)tile * FT * out_w;
        if (MODE == 0) {
            for (int i = tid; i < nf * NBP; i += FEAT_THREADS) orow[i] = ptile[i];
        } else {
            // Filterbank with the lanes of a warp over the frames of the tile and one edge
            // interval per lane group: the bins of interval j are walked once, giving
            // both their rising sum (band j) and their falling sum (band j-1); all lanes
            // of an interval walk the same bins (weights are broadcasts, the odd row
            // strides keep the other accesses conflict-free, no lane waits for a wider
            // band).  Band m = rising sum of interval m + falling sum of interval m+1,
            // added while the results are written out contiguously.
            float *up_s = reinterpret_cast<float *>(fbuf);            // [FT][M+1], transforms are done
            float *dn_s = up_s + FT * (M + 1);                        // [FT][M+1]
            const float2 *mw2 = reinterpret_cast<const float2 *>(mw);
            constexpr int BPW = 32 / FT;                              // intervals per warp step
            const int lane = tid & 31, warp = tid >> 5;
            const int f = lane % FT, sub = lane / FT;
            for (int j0 = warp * BPW; j0 <= M; j0 += (FEAT_THREADS / 32) * BPW) {
                const int j = j0 + sub;
                if (j <= M && f < nf) {
                    const float *p = ptile + f * NBP;
                    float u = 0.f, d = 0.f;
                    const int k1 = mst[j + 1];
                    for (int k = mst[j]; k < k1; ++k) {
                        const float2 w = mw2[k];
                        const float pk = p[k];
                        u = fmaf(w.x, pk, u);
                        d = fmaf(w.y, pk, d);
                    }
                    up_s[f * (M + 1) + j] = u;
                    dn_s[f * (M + 1) + j] = d;
                }
            }
            __syncthreads();
            // element i = frame * M + band sits at i + frame in the [FT][M+1] sums: walked without a division
            int ff = out_f0, m = out_m0;
            for (int i = tid; i < nf * M; i += FEAT_THREADS) {
                orow[i] = compress(up_s[i + ff] + dn_s[i + ff + 1], floor_v, comp);
                ff += step_f;
                m += step_m;
                if (m >= M) {
                    m -= M;
                    ++ff;
                }
            }
        }
        __syncthreads();   // ptile, the interval sums (= the transform buffers) and chunk are reused by the next tile
    }
}

// ---------------------------------------------------------------- fused path, one warp per frame pair
// 512-point transforms of the fused path.  A warp takes a frame pair from its
// samples to its two power spectra: lane t holds 16 of the 512 complex points
// (frame 2p in the real, frame 2p+1 in the imaginary part) as two radix-8
// butterflies per pass, exchanges them through a buffer of its own (warp barriers
// only), and in the last pass takes butterflies t and 64-t, whose outputs are the
// bins k and 512-k: the two spectra are separated and squared in registers and
// only the powers go to shared memory.  A CTA of eight warps does a tile of 16
// frames at a time; the filterbank then runs with the frames of the tile over the
// lanes (every edge interval walked once, all lanes on the same bins), while the
// samples of the next tile are already on their way from global memory.
namespace wp {

constexpr int K = 512;
constexpr int NBP = K / 2 + 1;
constexpr int XB = padded_points(K);          // float2 slots of a warp's exchange buffer
constexpr int WARPS = FEAT_THREADS / 32;
constexpr int FT = 2 * WARPS;                  // frames per tile: one pair per warp
constexpr int SV = 3;                          // 128-bit staging loads per thread, array and tile

template <int NS>
__device__ __forceinline__ void scatter8(const float2 *v, float2 *s, int j) {
    constexpr int PS = out_shift(NS);
    const int k = j & (NS - 1);
    const int base = padi<PS>((j - k) * 8 + k);
#pragma unroll
    for (int r = 0; r < 8; ++r) s[base + padi<PS>(r * NS)] = v[r];
}

// |A|^2 and |B|^2 at bin k from Z[k] = z and Z[K-k] = q, where Z is the transform of a + i b.
__device__ __forceinline__ void power_pair(float2 z, float2 q, float &pa, float &pb) {
    const float ar = z.x + q.x, ai = z.y - q.y;
    const float br = z.y + q.y, bi = z.x - q.x;
    pa = 0.25f * fmaf(ar, ar, ai * ai);
    pb = 0.25f * fmaf(br, br, bi * bi);
}

__host__ __device__ constexpr int chunk_floats(int win, int hop) { return ((FT - 1) * hop + win + 3) & ~3; }
__host__ __device__ constexpr size_t smem_bytes(int win, int hop, int M) {
    return sizeof(float2) * WARPS * XB + 3 * sizeof(float) * chunk_floats(win, hop) + sizeof(float) * K +
           sizeof(float2) * (NBP + 1) + sizeof(int) * (M + 2);
}

// Once a warp's transforms are done its exchange buffer (2 XB floats) holds the two
// power spectra of its frame pair and, behind them, the pair's interval sums.  Rows
// start at different banks so that the frames of a tile can be read side by side.
constexpr int ROW_SPAN = 2 * XB;                   // floats of a warp's buffer
constexpr int SUMS_OFF = 2 * NBP + 2 * WARPS;      // floats before the sums of a pair
__device__ __forceinline__ int power_row(int f) { return (f >> 1) * ROW_SPAN + (f & 1) * NBP + (f >> 1) * 2; }
// sums of frame f: [rising, falling][M + 1]
__device__ __forceinline__ int sums_row(int f, int M) {
    return (f >> 1) * ROW_SPAN + SUMS_OFF + (f >> 1) * 4 + (f & 1) * 2 * (M + 1);
}
static_assert(SUMS_OFF + 4 * WARPS + 4 * (aug::MAX_MEL + 1) <= ROW_SPAN, "sums fit behind the power rows");

// 16 bytes global -> shared without passing through registers; bytes = 0 stores zeros.
__device__ __forceinline__ void copy16_async(float *dst_smem, const float *src, int bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(
                     (unsigned)__cvta_generic_to_shared(dst_smem)),
                 "l"(src), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void copies_done() { asm volatile("cp.async.wait_all;" ::: "memory"); }

template <int TILES>
__global__ void __launch_bounds__(FEAT_THREADS, FEAT_MINB)
frames_warp_kernel(const float *__restrict__ in_a, const float *__restrict__ in_b, int64_t in_stride,
                   const float *__restrict__ gain, const int *__restrict__ lengths, int win, int hop,
                   int M, int T_max, const aug::MelBin *__restrict__ melw,
                   const int *__restrict__ melstart, const float2 *__restrict__ tw, float floor_v,
                   float pad_v, int comp, float *__restrict__ out, int *__restrict__ counts, int n_cap) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int chunk_cap = chunk_floats(win, hop);
    float2 *xb_all = reinterpret_cast<float2 *>(smem_raw);                   // [WARPS][XB]; later powers and sums
    float *prow = reinterpret_cast<float *>(xb_all);
    float *chunk = reinterpret_cast<float *>(xb_all + WARPS * XB);           // [chunk_cap] y_s + g v of the tile
    float *raw_a = chunk + chunk_cap;                                        // [chunk_cap] y_s of the next tile
    float *raw_b = raw_a + chunk_cap;                                        // [chunk_cap] v of the next tile
    float *win_s = raw_b + chunk_cap;                                        // [K] Hann, zero beyond win
    float2 *mw = reinterpret_cast<float2 *>(win_s + K);                      // [NBP + 1] (up, down)
    int *mst = reinterpret_cast<int *>(mw + NBP + 1);                        // [M + 2]

    const int utt = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int run0 = blockIdx.x * (FT * TILES);
    const int N = min(max(lengths[utt], 0), n_cap);
    const int T = min(frame_count(N, win, hop), T_max);
    if (blockIdx.x == 0 && tid == 0) counts[utt] = T;
    const int rows = min(FT * TILES, T_max - run0);
    if (rows <= 0) return;
    const int nfr = max(0, min(FT * TILES, T - run0));
    float *orun = out + ((int64_t)utt * T_max + run0) * M;
    for (int i = nfr * M + tid; i < rows * M; i += FEAT_THREADS) orun[i] = pad_v;
    if (nfr == 0) return;

    const float g = gain[utt];
    const float *ra = in_a + (int64_t)utt * in_stride;
    const float *rb = in_b + (int64_t)utt * in_stride;
    // 128-bit staging needs 16-byte aligned tile starts and at most SV loads per thread
    const bool vec = (hop & 3) == 0 && (in_stride & 3) == 0 && chunk_cap <= SV * FEAT_THREADS * 4;
    // 64-bit loads of sample pairs: frames start on even samples and the window ends on one
    const bool pairs = ((hop | win) & 1) == 0 && win >= 2;
    for (int n = tid; n < K; n += FEAT_THREADS)
        win_s[n] = n < win ? 0.5f - 0.5f * cospif(2.f * (float)n / (float)win) : 0.f;
    for (int k = tid; k < NBP; k += FEAT_THREADS) {
        const aug::MelBin w = melw[(int64_t)utt * NBP + k];
        mw[k] = make_float2(w.up, w.down);
    }
    for (int m = tid; m < M + 2; m += FEAT_THREADS) mst[m] = melstart[(int64_t)utt * (M + 2) + m];

    // Lane constants: twiddles of the last pass for this lane's two butterflies
    // (j0 = lane and its mirror j1 = 64 - lane; lane 0 takes the self-mirrored 0 and 32)
    // and the first twiddle of the middle pass.
    const int j0 = lane, j1 = lane ? 64 - lane : 32;
    float2 w3a[8], w3b[8];
    twiddle_powers<8>(w3a, __ldg(&tw[tw_index(K, j0)]));
    twiddle_powers<8>(w3b, __ldg(&tw[tw_index(K, j1)]));
    const float2 w2_1 = __ldg(&tw[tw_index(64, lane & 7)]);
    float2 *xb = xb_all + warp * XB;
    const int n_tiles = min(TILES, (nfr + FT - 1) / FT);
    const int out_f0 = tid / M, out_m0 = tid - out_f0 * M;                   // first output element of this thread
    const int step_f = FEAT_THREADS / M, step_m = FEAT_THREADS - step_f * M;  // and the stride to its next one

    // Samples of a tile travel global -> shared asynchronously, one tile ahead: a thread
    // copies the 16-byte groups i = 4 (tid + 256 u) of y_s and v into raw_a / raw_b, and
    // one tile later mixes the same groups into `chunk`, so the raw slots are private to
    // the thread and need no barrier; groups beyond the tile's stretch are zero-filled.
    auto stage_issue = [&](int tile) {
        const int s0 = (run0 + tile * FT) * hop;
        const int ns = (min(FT, T - (run0 + tile * FT)) - 1) * hop + win;
#pragma unroll
        for (int u = 0; u < SV; ++u) {
            const int i = (tid + u * FEAT_THREADS) * 4;
            if (i < chunk_cap) {
                // rows are allocated up to a multiple of 4 floats: whole groups can be read
                const int ok = i < ns ? 16 : 0;
                const int isrc = ok ? s0 + i : 0;
                copy16_async(raw_a + i, ra + isrc, ok);
                if (g != 0.f) copy16_async(raw_b + i, rb + isrc, ok);
            }
        }
    };
    auto stage_mix = [&]() {
#pragma unroll
        for (int u = 0; u < SV; ++u) {
            const int i = (tid + u * FEAT_THREADS) * 4;
            if (i < chunk_cap) {
                float4 x = *reinterpret_cast<const float4 *>(raw_a + i);
                if (g != 0.f) {
                    const float4 y = *reinterpret_cast<const float4 *>(raw_b + i);
                    x = make_float4(fmaf(g, y.x, x.x), fmaf(g, y.y, x.y), fmaf(g, y.z, x.z), fmaf(g, y.w, x.w));
                }
                *reinterpret_cast<float4 *>(chunk + i) = x;
            }
        }
    };
    auto stage_scalar = [&](int tile) {
        const int s0 = (run0 + tile * FT) * hop;
        const int ns = (min(FT, T - (run0 + tile * FT)) - 1) * hop + win;
        for (int i = tid; i < ns; i += FEAT_THREADS)
            chunk[i] = g != 0.f ? fmaf(g, rb[s0 + i], ra[s0 + i]) : ra[s0 + i];
        for (int i = ns + tid; i < chunk_cap; i += FEAT_THREADS) chunk[i] = 0.f;
    };
    if (vec) stage_issue(0);

    for (int tile = 0; tile < n_tiles; ++tile) {
        const int t0 = run0 + tile * FT;
        const int nf = min(FT, T - t0);
        if (vec) {
            copies_done();
            stage_mix();
            if (tile + 1 < n_tiles) stage_issue(tile + 1);
        } else {
            stage_scalar(tile);
        }
        __syncthreads();                      // chunk (and, first time, the tables) in place; sums of the last tile read

        const int f0 = 2 * warp;
        if (f0 < nf) {
            const bool have1 = f0 + 1 < nf;
            const float *c0 = chunk + f0 * hop;
            float2 v[2][8];
            if (pairs) {
                // First pass on butterflies j = 2 lane and 2 lane + 1 (points j + 64 r): adjacent
                // samples, one 64-bit load each from the window table and the two frames.  A point
                // beyond the window reads the window's last pair instead (its weight is zero).
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    const int n = 2 * lane + 64 * r;
                    const int nc = min(n, win - 2);
                    const float2 wn = *reinterpret_cast<const float2 *>(win_s + n);
                    const float2 a = *reinterpret_cast<const float2 *>(c0 + nc);
                    const float2 bb = *reinterpret_cast<const float2 *>(c0 + hop + nc);
                    v[0][r] = make_float2(wn.x * a.x, wn.x * bb.x);
                    v[1][r] = make_float2(wn.y * a.y, wn.y * bb.y);
                }
            } else {
#pragma unroll
                for (int b = 0; b < 2; ++b) {
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        const int n = 2 * lane + b + 64 * r;
                        float a = 0.f, bb = 0.f;
                        if (n < win) {
                            const float wn = win_s[n];
                            a = wn * c0[n];
                            if (have1) bb = wn * c0[hop + n];
                        }
                        v[b][r] = make_float2(a, bb);
                    }
                }
            }
            Dft<8>::run(v[0]);
            Dft<8>::run(v[1]);
            scatter8<1>(v[0], xb, 2 * lane);
            scatter8<1>(v[1], xb, 2 * lane + 1);
            __syncwarp();
            gather<K, 16, 8, 1>(v, xb, lane);
            __syncwarp();
            {
                float2 w2[8];
                twiddle_powers<8>(w2, w2_1);
#pragma unroll
                for (int r = 1; r < 8; ++r) {
                    v[0][r] = cmul(v[0][r], w2[r]);
                    v[1][r] = cmul(v[1][r], w2[r]);
                }
            }
            Dft<8>::run(v[0]);
            Dft<8>::run(v[1]);
            scatter8<8>(v[0], xb, lane);
            scatter8<8>(v[1], xb, lane + 32);
            __syncwarp();
            {
                constexpr int PS = out_shift(8);
                const int b0 = padi<PS>(j0), b1 = padi<PS>(j1);
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    v[0][r] = xb[b0 + padi<PS>(r * 64)];
                    v[1][r] = xb[b1 + padi<PS>(r * 64)];
                }
            }
#pragma unroll
            for (int r = 1; r < 8; ++r) {
                v[0][r] = cmul(v[0][r], w3a[r]);
                v[1][r] = cmul(v[1][r], w3b[r]);
            }
            Dft<8>::run(v[0]);     // bins j0 + 64 r
            Dft<8>::run(v[1]);     // bins j1 + 64 r
            // Bin k pairs with bin 512 - k: for j0 + 64 r that is output 7 - r of the other
            // butterfly (lane 0: butterfly 0 pairs with itself, 64 r with 64 (8 - r), and so
            // does butterfly 32).  Only bins up to 256 are kept.
            __syncwarp();                     // every lane has its last-pass inputs: the buffer is free
            float *p0 = prow + power_row(f0), *p1 = prow + power_row(f0 + 1);
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float2 qa = lane ? v[1][7 - r] : v[0][(8 - r) & 7];
                const float2 qb = lane ? v[0][7 - r] : v[1][7 - r];
                float pa, pb;
                power_pair(v[0][r], qa, pa, pb);
                p0[j0 + 64 * r] = pa;
                if (have1) p1[j0 + 64 * r] = pb;
                power_pair(v[1][r], qb, pa, pb);
                p0[j1 + 64 * r] = pa;
                if (have1) p1[j1 + 64 * r] = pb;
            }
            if (lane == 0) {
                float pa, pb;
                power_pair(v[0][4], v[0][4], pa, pb);
                p0[K / 2] = pa;
                if (have1) p1[K / 2] = pb;
            }
        }
        __syncthreads();                      // power spectra of the tile in place

        // Filterbank with the frames of the tile over the lanes, two adjacent edge
        // intervals per warp step: the bins of interval j give its rising sum (band j) and
        // its falling sum (band j-1).  Intervals widen with frequency, so the pairs are
        // dealt to the warps from the widest down, back and forth, which evens out the
        // bins each warp walks.
        {
            const int f = lane & (FT - 1), sub = lane / FT;
            static_assert(FT == 16, "two intervals per warp step");
            const int npairs = (M + 2) / 2;                  // intervals 0 .. M in pairs (2q, 2q+1)
            for (int st = 0; st * WARPS < npairs; ++st) {
                const int q = npairs - 1 - (st * WARPS + ((st & 1) ? WARPS - 1 - warp : warp));
                const int j = 2 * q + sub;
                if (q >= 0 && j <= M && f < nf) {
                    const float *p = prow + power_row(f);
                    float u0 = 0.f, d0 = 0.f, u1 = 0.f, d1 = 0.f;
                    int k = mst[j];
                    const int k1 = mst[j + 1];
                    for (; k + 1 < k1; k += 2) {
                        const float2 wa = mw[k], wb = mw[k + 1];
                        const float pa = p[k], pb = p[k + 1];
                        u0 = fmaf(wa.x, pa, u0);
                        d0 = fmaf(wa.y, pa, d0);
                        u1 = fmaf(wb.x, pb, u1);
                        d1 = fmaf(wb.y, pb, d1);
                    }
                    if (k < k1) {
                        const float2 wa = mw[k];
                        const float pa = p[k];
                        u0 = fmaf(wa.x, pa, u0);
                        d0 = fmaf(wa.y, pa, d0);
                    }
                    float *sm = prow + sums_row(f, M);
                    sm[j] = u0 + u1;
                    sm[M + 1 + j] = d0 + d1;
                }
            }
        }
        __syncthreads();                      // interval sums in place
        float *orow = orun + (int64_t)tile * FT * M;
        {
            // element i = frame * M + band, walked without a division
            int ff = out_f0, m = out_m0;
            for (int i = tid; i < nf * M; i += FEAT_THREADS) {
                const float *sm = prow + sums_row(ff, M);
                const float e = fmaxf(sm[m] + sm[M + 1 + m + 1], floor_v);
                const float l = __logf(e);
                orow[i] = comp == AUG_COMPRESS_LOG ? l : __expf(l * (1.f / 15.f));
                ff += step_f;
                m += step_m;
                if (m >= M) {
                    m -= M;
                    ++ff;
                }
            }
        }
    }
}

}  // namespace wp

// ---------------------------------------------------------------- step 4 alone
__global__ void __launch_bounds__(256)
logmel_kernel(const float *__restrict__ power, const int *__restrict__ counts, int NBP, int M,
              int T_max, const aug::MelBin *__restrict__ melw, const int *__restrict__ melstart,
              float floor_v, float pad_v, int comp, float *__restrict__ feats) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    aug::MelBin *mw = reinterpret_cast<aug::MelBin *>(smem_raw);
    int *mst = reinterpret_cast<int *>(mw + NBP + 1);
    const int utt = blockIdx.y, tid = threadIdx.x;
    constexpr int FT = 8;
    const int t0 = blockIdx.x * FT;
    const int rows = min(FT, T_max - t0);
    if (rows <= 0) return;
    const int T = min(max(counts[utt], 0), T_max);
    for (int k = tid; k < NBP; k += 256) mw[k] = melw[(int64_t)utt * NBP + k];
    for (int m = tid; m < M + 2; m += 256) mst[m] = melstart[(int64_t)utt * (M + 2) + m];
    __syncthreads();
    for (int i = tid; i < rows * M; i += 256) {
        const int f = i / M, m = i - f * M, t = t0 + f;
        float val = pad_v;
        if (t < T)
            val = compress(band_energy(power + ((int64_t)utt * T_max + t) * NBP, mw, mst, m),
                           floor_v, comp);
        feats[((int64_t)utt * T_max + t) * M + m] = val;
    }
}

template <int K, int MODE>
int launch_frames(AugCtx *ctx, const float *a, const float *b, int64_t stride, const int *lengths,
                  const AugUttParams *table, int B, float *out, int T_max, int *counts, int n_cap) {
    const AugConfig &c = ctx->cfg;
    constexpr int FT = Plan<K>::FT, NBP = K / 2 + 1;
    const int chunk_cap = ((FT - 1) * c.hop + c.win + 3) & ~3;
    const size_t smem = sizeof(float) * fbuf_floats<K>(FT, c.n_mel) + sizeof(float) * FT * NBP +
                        sizeof(float) * chunk_cap + sizeof(aug::MelBin) * (NBP + 1) +
                        sizeof(int) * (c.n_mel + 2);
    if (smem > 227 * 1024) return AUG_ECAP;
    // A CTA works through a run of tiles (window values, filterbank tables and other
    // set-up once per run) unless the batch is so small that single tiles are needed
    // to give every multiprocessor something to do.
    const int n_tiles = (T_max + FT - 1) / FT;
    const bool runs = (int64_t)n_tiles * B >= 2 * (int64_t)ctx->sm_count * Plan<K>::TILES;
    const int RUN = FT * (runs ? Plan<K>::TILES : 1);
    dim3 grid((T_max + RUN - 1) / RUN, B);
    auto kern = runs ? frames_kernel<K, MODE, Plan<K>::TILES> : frames_kernel<K, MODE, 1>;
    if ((runs ? smem_opt_in<frames_kernel<K, MODE, Plan<K>::TILES>>(ctx->device)
              : smem_opt_in<frames_kernel<K, MODE, 1>>(ctx->device)) != AUG_OK)
        return AUG_ECUDA;
    kern<<<grid, FEAT_THREADS, smem, ctx->stream>>>(
        a, b, stride, ctx->gain, table, lengths, c.win, c.hop, c.n_mel, T_max, ctx->melw,
        ctx->melstart, ctx->tw, c.log_floor, c.pad_value, c.compression, out, counts,
        n_cap);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

}  // namespace

int launch_mel_tables(AugCtx *ctx, const AugUttParams *table, int B, cudaStream_t st) {
    const AugConfig &c = ctx->cfg;
    mel_tables_kernel<<<B, 256, 0, st>>>(table, c.n_fft, c.n_mel, (double)c.fs,
                                                  (double)c.f_lo, (double)c.f_hi, ctx->melw,
                                                  ctx->melstart, c.vtlp_win > 0 ? 1 : 0);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

int launch_stft_power(AugCtx *ctx, const float *wave, int64_t stride, const int *lengths, int B,
                      float *power, int T_max, int *counts) {
    if (T_max <= 0) return AUG_OK;
    const int n_cap = (int)(stride < 0x7fffffff ? stride : 0x7fffffff);     // the caller's rows end at their stride
    if (ctx->cfg.n_fft == 512)
        return launch_frames<512, 0>(ctx, wave, nullptr, stride, lengths, nullptr, B, power, T_max, counts, n_cap);
    return launch_frames<1024, 0>(ctx, wave, nullptr, stride, lengths, nullptr, B, power, T_max, counts, n_cap);
}

#ifndef FEAT_WP_TILES
#define FEAT_WP_TILES 8     // consecutive 16-frame tiles one CTA of the warp-per-pair kernel works through
#endif

// Fused features with the 512-point transform: the warp-per-frame-pair kernel.
static int launch_frames_warp(AugCtx *ctx, const int *lengths, int B, float *feats, int T_max, int *counts,
                              int max_len) {
    const AugConfig &c = ctx->cfg;
    const size_t smem = wp::smem_bytes(c.win, c.hop, c.n_mel);
    if (smem > 227 * 1024) return AUG_ECAP;
    const int n_tiles = (T_max + wp::FT - 1) / wp::FT;
    const bool runs = (int64_t)n_tiles * B >= 2 * (int64_t)ctx->sm_count * FEAT_WP_TILES;
    const int RUN = wp::FT * (runs ? FEAT_WP_TILES : 1);
    dim3 grid((T_max + RUN - 1) / RUN, B);
    auto kern = runs ? wp::frames_warp_kernel<FEAT_WP_TILES> : wp::frames_warp_kernel<1>;
    if ((runs ? smem_opt_in<wp::frames_warp_kernel<FEAT_WP_TILES>>(ctx->device)
              : smem_opt_in<wp::frames_warp_kernel<1>>(ctx->device)) != AUG_OK)
        return AUG_ECUDA;
    kern<<<grid, FEAT_THREADS, smem, ctx->stream>>>(
        ctx->ys, ctx->vv, ctx->ws_stride, ctx->gain, lengths, c.win, c.hop, c.n_mel, T_max, ctx->melw,
        ctx->melstart, ctx->tw, c.log_floor, c.pad_value, c.compression, feats, counts, max_len);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

// max_len: the length clamp the convolution used, so that every stage cuts an over-long
// entry of `lengths` at the same sample.
int launch_fused_features(AugCtx *ctx, const int *lengths, const AugUttParams *table, int B,
                          float *feats, int T_max, int *counts, int max_len) {
    if (T_max <= 0) return AUG_OK;
#ifndef FEAT_OLD_512
    if (ctx->cfg.n_fft == 512) return launch_frames_warp(ctx, lengths, B, feats, T_max, counts, max_len);
#endif
    if (ctx->cfg.n_fft == 512)
        return launch_frames<512, 1>(ctx, ctx->ys, ctx->vv, ctx->ws_stride, lengths, table, B, feats,
                                     T_max, counts, max_len);
    return launch_frames<1024, 1>(ctx, ctx->ys, ctx->vv, ctx->ws_stride, lengths, table, B, feats,
                                  T_max, counts, max_len);
}

int launch_logmel(AugCtx *ctx, const float *power, const int *counts, int B, int T_max,
                  float *feats) {
    const AugConfig &c = ctx->cfg;
    if (T_max <= 0) return AUG_OK;
    const int NBP = ctx->n_bins;
    const size_t smem = sizeof(aug::MelBin) * (NBP + 1) + sizeof(int) * (c.n_mel + 2);
    dim3 grid((T_max + 7) / 8, B);
    logmel_kernel<<<grid, 256, smem, ctx->stream>>>(power, counts, NBP, c.n_mel, T_max, ctx->melw,
                                                    ctx->melstart, c.log_floor, c.pad_value,
                                                    c.compression, feats);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}

// ---------------------------------------------------------------- step 4 without any allocation
//
// feat_vtlp_logmel needs two small per-utterance tables (filterbank weights per
// DFT bin, first bin of every band interval) that normally live in the context's
// workspace, and a context cannot exist without cudaMalloc.  Some callers are not
// allowed to allocate: a plug-in running inside a host application that has
// handed every byte of device memory to its own pool, a real-time feature
// front-end that must not touch the allocator after start-up, or code that only
// receives device pointers and a stream.  For them the tables live in a
// fixed-size array that is part of the loaded library image, so nothing is
// allocated at call time -- at the price that every GPU that loads the library
// carries the array until the process exits, and that all calls share it.
namespace {

constexpr int NOALLOC_BINS = 513;                                   // n_fft <= 1024
constexpr size_t NOALLOC_MELW_BYTES =
    sizeof(aug::MelBin) * (size_t)AUG_NOALLOC_MAX_BATCH * NOALLOC_BINS;          // 1 050 624
constexpr size_t NOALLOC_START_BYTES =
    sizeof(int) * (size_t)AUG_NOALLOC_MAX_BATCH * (aug::MAX_MEL + 2);            //   133 120
static_assert(NOALLOC_MELW_BYTES % 256 == 0, "second table must stay 256-byte aligned");

// The scratch itself.  In host code this name is only a handle for the runtime,
// not an address a kernel could use; the device address is looked up below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_MELW_BYTES + NOALLOC_START_BYTES];

constexpr int NOALLOC_MAX_DEVICES = 64;
void *g_noalloc_addr[NOALLOC_MAX_DEVICES];   // device address of the scratch, per device; NULL = not looked up yet

// Device address of the scratch on the current device.  The first call on a
// device asks the runtime for it (no allocation: the array already exists in the
// module); later calls reuse the cached pointer.
int noalloc_scratch(void **out) {
    int dev = -1;
    AUG_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return AUG_ECAP;
    void *p = __atomic_load_n(&g_noalloc_addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        AUG_CUDA_OK(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        if (!p) return AUG_ECUDA;
        __atomic_store_n(&g_noalloc_addr[dev], p, __ATOMIC_RELEASE);   // same value from any thread
    }
    *out = p;
    return AUG_OK;
}

}  // namespace

extern "C" int feat_vtlp_logmel_noalloc(const AugConfig *cfg, const float *power_dev,
                                        const int *frame_counts_dev,
                                        const AugUttParams *table_dev, int B, int T_max,
                                        float *feats_dev, void *cuda_stream) {
    if (!cfg || !power_dev || !frame_counts_dev || !table_dev || !feats_dev) return AUG_EINVAL;
    if (B < 0 || T_max <= 0) return AUG_EINVAL;
    if (cfg->n_fft != 512 && cfg->n_fft != 1024) return AUG_EINVAL;
    if (cfg->n_mel < 1 || cfg->fs <= 0 || !(cfg->f_lo >= 0.f) || !(cfg->f_hi > cfg->f_lo) ||
        cfg->f_hi > 0.5f * cfg->fs + 1e-3f || !(cfg->log_floor > 0.f) || !isfinite(cfg->pad_value))
        return AUG_EINVAL;
    if (cfg->compression != AUG_COMPRESS_LOG && cfg->compression != AUG_COMPRESS_POW_1_15)
        return AUG_EINVAL;
    // the fixed scratch holds tables for this many utterances and bands, no more
    if (B > AUG_NOALLOC_MAX_BATCH || cfg->n_mel > aug::MAX_MEL) return AUG_ECAP;
    if (B == 0) return AUG_OK;

    void *scratch = nullptr;
    int rc = noalloc_scratch(&scratch);
    if (rc != AUG_OK) return rc;
    aug::MelBin *melw = reinterpret_cast<aug::MelBin *>(scratch);
    int *melstart = reinterpret_cast<int *>(static_cast<unsigned char *>(scratch) + NOALLOC_MELW_BYTES);

    // Both tables are written in full for utterances [0, B) before they are read
    // (same stream), so nothing left by an earlier call is ever seen and nothing
    // needs clearing.
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int nbp = cfg->n_fft / 2 + 1;
    mel_tables_kernel<<<B, 256, 0, st>>>(table_dev, cfg->n_fft, cfg->n_mel, (double)cfg->fs,
                                         (double)cfg->f_lo, (double)cfg->f_hi, melw, melstart, 0);
    AUG_CUDA_OK(cudaGetLastError());
    const size_t smem = sizeof(aug::MelBin) * (nbp + 1) + sizeof(int) * (cfg->n_mel + 2);
    dim3 grid((T_max + 7) / 8, B);
    logmel_kernel<<<grid, 256, smem, st>>>(power_dev, frame_counts_dev, nbp, cfg->n_mel, T_max,
                                           melw, melstart, cfg->log_floor, cfg->pad_value,
                                           cfg->compression, feats_dev);
    AUG_CUDA_OK(cudaGetLastError());
    return AUG_OK;
}
