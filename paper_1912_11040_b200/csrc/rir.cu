// Step 1: room impulse responses by the image-source method.
//
// One CTA builds one impulse response (one utterance, one source) in shared
// memory.  Geometry runs in fp64, once per image and spread over the lanes of a
// warp; the 2*W_h+1 taps of each image are then spread over the lanes in fp32:
// with tau = n0 + phi, sin(pi (n - tau)) = -(-1)^(n-n0) sin(pi phi), so a tap costs
// one division and a few FMAs, and the Hann factor comes from the angle-sum
// identity with per-lane constants.  The lattice points with |kx|+|ky|+|kz| <= order
// are enumerated compactly (a prefix over kx, then closed forms inside the diamond
// of (ky, kz)), so every lane of a warp carries a real image.
#include "common.cuh"

namespace {

#ifndef RIR_THREADS_N
#define RIR_THREADS_N 1024
#endif
constexpr int RIR_THREADS = RIR_THREADS_N;
constexpr int AX = 2 * aug::MAX_ORDER + 1;

__device__ __forceinline__ double ipow(double b, int e) {
    double r = 1.0;
    for (int i = 0; i < e; ++i) r *= b;
    return r;
}

__global__ void __launch_bounds__(RIR_THREADS)
rir_image_kernel(const AugUttParams *__restrict__ table, int S_max, int L, int half_w, double fs,
                 double c, int max_order, int cube, float *__restrict__ rir, int *status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *dsq = reinterpret_cast<double *>(smem_raw);   // [3][AX]
    double *gain = dsq + 3 * AX;                          // [3][AX]
    int *xpre = reinterpret_cast<int *>(gain + 3 * AX);   // [AX + 1] images before slab kx
    float *h = reinterpret_cast<float *>(xpre + AX + 3);  // [L]

    const int utt = blockIdx.y, s = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const AugUttParams &row = table[utt];
    float *out = rir + ((int64_t)utt * S_max + s) * L;

    const int n_src = row.n_src, order = row.order;
    int bad = 0;
    if (n_src < 1 || n_src > S_max) bad = aug::R_NSRC;
    else if (order < 0 || order > max_order) bad = aug::R_ORDER;
    if (bad || s >= n_src) {
        for (int i = tid; i < L; i += RIR_THREADS) out[i] = 0.f;
        if (bad && tid == 0 && s == 0) {
            if (atomicCAS(&status[0], -1, utt) == -1) status[1] = bad;
        }
        return;
    }

    for (int i = tid; i < L; i += RIR_THREADS) h[i] = 0.f;
    const int side = 2 * order + 1;
    if (tid < 3 * side) {
        const int a = tid / side, k = tid % side - order;
        const int p = k & 1;            // k = 2m - p
        const int m = (k + p) / 2;
        const double img = (1 - 2 * p) * (double)row.src_pos[s][a] + 2.0 * m * (double)row.room[a];
        const double diff = img - (double)row.mic[a];
        dsq[a * AX + k + order] = diff * diff;
        gain[a * AX + k + order] = ipow((double)row.beta[2 * a], abs(m - p)) *
                                   ipow((double)row.beta[2 * a + 1], abs(m));
    }
    if (tid == 0) {
        int run = 0;
        for (int ix = 0; ix < side; ++ix) {
            const int r = order - abs(ix - order);
            xpre[ix] = run;
            run += 2 * r * r + 2 * r + 1;      // points of the diamond |ky|+|kz| <= r
        }
        xpre[side] = run;
    }
    __syncthreads();
    const int total = cube ? side * side * side : xpre[side];

    // per-lane tap constants: this lane owns taps j = lane + 32 i - half_w
    float cj[3], sj[3], sg[3];
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        const int j = lane + 32 * i - half_w;
        cj[i] = cospif((float)j / (float)half_w);
        sj[i] = sinpif((float)j / (float)half_w);
        sg[i] = (j & 1) ? -1.f : 1.f;
    }
    const float fhw = (float)half_w;
    constexpr int NW = RIR_THREADS / 32;

    for (int base = warp * 32; base < total; base += NW * 32) {
        const int idx = base + lane;
        bool valid = idx < total;
        int n0 = 0;
        float phi = 0.f, A = 0.f, As = 0.f, cph = 0.f, sph = 0.f;
        if (valid) {
            int ix, ky, kz;
            if (cube) {
                ix = idx / (side * side);
                const int rem = idx - ix * side * side;
                ky = rem / side - order;
                kz = rem % side - order;
            } else {
                // slab kx: the last ix with xpre[ix] <= idx
                int lo = 0, hi = side;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (xpre[mid] <= idx) lo = mid; else hi = mid;
                }
                ix = lo;
                const int r = order - abs(ix - order);
                int q = idx - xpre[ix];               // position inside the diamond of radius r
                // rows ky = -r..0 hold 1, 3, .., 2r+1 points (q < (r+1)^2, row u has u^2 before it);
                // rows ky = 1..r mirror rows r-1..0, counted from the end.
                const bool upper = q >= (r + 1) * (r + 1);
                if (upper) q = 2 * r * r + 2 * r - q;
                int u = (int)sqrtf((float)q);
                if (u * u > q) --u;
                if ((u + 1) * (u + 1) <= q) ++u;
                ky = upper ? r - u : u - r;
                kz = q - u * u - u;
            }
            const int iy = ky + order, iz = kz + order;
            {
                const double d = sqrt(dsq[ix] + dsq[AX + iy] + dsq[2 * AX + iz]);
                const double g = gain[ix] * gain[AX + iy] * gain[2 * AX + iz];
                const double tau = d * fs / c;
                const double rt = rint(tau);
                A = (float)(g / d);
                valid = (A != 0.f) && (rt - half_w < (double)L);
                n0 = (int)rt;
                phi = (float)(tau - rt);
                As = -A * sinpif(phi) * 0.318309886183790671538f;
                cph = 0.5f * cospif(phi / fhw);
                sph = 0.5f * sinpif(phi / fhw);
            }
        }
        unsigned mask = __ballot_sync(0xffffffffu, valid);
        while (mask) {
            const int src = __ffs(mask) - 1;
            mask &= mask - 1;
            const int n0b = __shfl_sync(0xffffffffu, n0, src);
            const float phib = __shfl_sync(0xffffffffu, phi, src);
            const float Ab = __shfl_sync(0xffffffffu, A, src);
            const float Asb = __shfl_sync(0xffffffffu, As, src);
            const float cb = __shfl_sync(0xffffffffu, cph, src);
            const float sb = __shfl_sync(0xffffffffu, sph, src);
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const int jj = lane + 32 * i;
                const int j = jj - half_w;
                const int n = n0b + j;
                const float x = (float)j - phib;
                if (jj <= 2 * half_w && (unsigned)n < (unsigned)L && fabsf(x) <= fhw) {
                    const float hann = 0.5f + cj[i] * cb + sj[i] * sb;
                    const float sc = (fabsf(x) < 1e-7f) ? Ab : __fdividef(sg[i] * Asb, x);
                    atomicAdd(&h[n], sc * hann);
                }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < L; i += RIR_THREADS) out[i] = h[i];
}

}  // namespace

int launch_rir(AugCtx *ctx, const AugUttParams *table, int B, float *rir, cudaStream_t st) {
    const AugConfig &c = ctx->cfg;
    const size_t smem = sizeof(double) * 6 * AX + sizeof(int) * (AX + 3) + sizeof(float) * (size_t)c.rir_taps;
    // (set on every launch: the attribute belongs to the current device's copy of the kernel)
    AUG_CUDA_OK(cudaFuncSetAttribute(rir_image_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem));
    dim3 grid(c.max_sources, B);
    rir_image_kernel<<<grid, RIR_THREADS, smem, st>>>(
        table, c.max_sources, c.rir_taps, c.frac_half_width, (double)c.fs, (double)c.sound_speed,
        c.max_order, c.image_lattice == AUG_LATTICE_CUBE ? 1 : 0, rir, ctx->status);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}
