// Step 1: room impulse responses by the image-source method.
//
// One CTA builds one impulse response (one utterance, one source) in shared
// memory.  Every warp works through batches of 32 images in two phases:
//
//   A  one image per lane: lattice point, distance and delay in fp64 (the delay
//      reaches 2.4e4 samples, where one fp32 ulp is 2e-3 samples), split into
//      an integer n0 and a fraction phi; the five numbers the taps need are
//      written, compacted over the images that contribute, to a slot of a small
//      shared-memory ring owned by the warp.
//   B  one image at a time, its 2 W_h + 1 taps over the lanes: lane l owns taps
//      l, l + 32, l + 64, so everything that depends only on the tap (its offset,
//      the cosine and sine of its Hann angle, its sign) sits in registers, and
//      the image's numbers arrive with two broadcast loads.  With tau = n0 + phi,
//      sin(pi (n - tau)) = -(-1)^(n - n0) sin(pi phi), and the Hann factor follows
//      from the angle-sum identity, so a tap costs one reciprocal, three FMAs
//      and one shared-memory reduction.
//
// The response is accumulated in 32-bit fixed point: a shared-memory fp32 atomic
// add is a compare-and-swap loop on this hardware, an integer one is a single
// instruction.  The scale is a power of two chosen per response from the direct
// path, the largest single contribution (A0 = 1/d0): full scale is 64 A0, one
// step 3e-8 A0 (coarser steps show in narrow mel bands that fall into a notch of
// the room's transfer function).  Integer sums are exact, so only the final value
// of a sample has to fit: with fully reflecting walls and order 32 the largest
// sample is 2-3 A0 in rooms of a few metres and 14 A0 in a 30 cm box; a sample
// beyond 64 A0 (rooms of a few centimetres) would wrap.
//
// The lattice points with |kx|+|ky|+|kz| <= order are enumerated compactly (a
// prefix over kx, then closed forms inside the diamond of (ky, kz)), so every
// lane of a warp carries a real image.
#include "common.cuh"

namespace {

constexpr int AX = 2 * aug::MAX_ORDER + 1;

__device__ __forceinline__ double ipow(double b, int e) {
    double r = 1.0;
    for (int i = 0; i < e; ++i) r *= b;
    return r;
}

__device__ __forceinline__ float rcp_approx(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// Add iv to the int at shared address a + OFF (one instruction, no result wanted).
template <int OFF>
__device__ __forceinline__ void red_shared_add(unsigned a, int iv) {
    asm volatile("red.shared.add.s32 [%0+%1], %2;" : : "r"(a), "n"(OFF), "r"(iv) : "memory");
}

// Bytes of dynamic shared memory of a CTA of `threads` threads for responses of L taps.
__host__ __device__ constexpr size_t rir_smem_bytes(int threads, int L) {
    return sizeof(double) * 3 * AX + sizeof(float) * 3 * AX + sizeof(int) * (AX + 3) +
           sizeof(float4) * threads + sizeof(float) * threads + sizeof(float) * (size_t)((L + 3) & ~3);
}

#ifndef RIR_THREADS
#define RIR_THREADS 512
#endif
#ifndef RIR_MINB
#define RIR_MINB 3
#endif
constexpr int THREADS = RIR_THREADS;      // 16 warps; two or three CTAs per multiprocessor
constexpr float HEADROOM_LOG2 = 6.f;   // full scale = 2^6 times the direct-path amplitude

__global__ void __launch_bounds__(THREADS, RIR_MINB)
rir_image_kernel(const AugUttParams *__restrict__ table, int S_max, int L, int half_w,
                 double fs_over_c, int max_order, int cube, float *__restrict__ rir, int *status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float4 *ring4 = reinterpret_cast<float4 *>(smem_raw);          // [THREADS] n0, phi, P0, P1 of an image
    int *h = reinterpret_cast<int *>(ring4 + THREADS);             // [L rounded up to 4] fixed-point response
    double *dsq = reinterpret_cast<double *>(h + ((L + 3) & ~3));  // [3][AX] squared coordinate differences
    float *ring1 = reinterpret_cast<float *>(dsq + 3 * AX);        // [THREADS] P2
    float *gain = ring1 + THREADS;                                 // [3][AX] wall gains per axis
    int *xpre = reinterpret_cast<int *>(gain + 3 * AX);            // [AX + 1] images before slab kx

    const int utt = blockIdx.y, s = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const AugUttParams &row = table[utt];
    float *out = rir + ((int64_t)utt * S_max + s) * L;

    const int n_src = row.n_src, order = row.order;
    int bad = 0;
    if (n_src < 1 || n_src > S_max) bad = aug::R_NSRC;
    else if (order < 0 || order > max_order) bad = aug::R_ORDER;
    if (bad || s >= n_src) {
        for (int i = tid; i < L; i += THREADS) out[i] = 0.f;
        if (bad && tid == 0 && s == 0) {
            if (atomicCAS(&status[0], -1, utt) == -1) status[1] = bad;
        }
        return;
    }

    for (int i = tid; i < ((L + 3) >> 2); i += THREADS) reinterpret_cast<int4 *>(h)[i] = make_int4(0, 0, 0, 0);
    const int side = 2 * order + 1;
    if (tid < 3 * side) {
        const int a = tid / side, k = tid % side - order;
        const int p = k & 1;            // k = 2m - p
        const int m = (k + p) / 2;
        const double img = (1 - 2 * p) * (double)row.src_pos[s][a] + 2.0 * m * (double)row.room[a];
        const double diff = img - (double)row.mic[a];
        dsq[a * AX + k + order] = diff * diff;
        gain[a * AX + k + order] = (float)(ipow((double)row.beta[2 * a], abs(m - p)) *
                                           ipow((double)row.beta[2 * a + 1], abs(m)));
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
    // fixed-point scale: a power of two with 2^31 / scale >= 2^HEADROOM_LOG2 / d0
    const float d0sq = (float)(dsq[order] + dsq[AX + order] + dsq[2 * AX + order]);
    const float e2 = d0sq > 0.f ? floorf(31.f - HEADROOM_LOG2 + 0.5f * log2f(d0sq)) : 0.f;
    const float scale = exp2f(fminf(fmaxf(e2, -60.f), 60.f)), inv_scale = exp2f(-fminf(fmaxf(e2, -60.f), 60.f));

    // Per-lane tap constants: this lane owns taps j = lane + 32 i - half_w, i < 3.  The
    // sign (-1)^j is the same for all three and is folded into the Hann constants; a
    // tap beyond 2 half_w gets an offset no window reaches.
    const float fhw = (float)half_w;
    const float sgn = ((lane - half_w) & 1) ? -1.f : 1.f;
    float fj[3], cj[3], sj[3];
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        const int jj = lane + 32 * i, j = jj - half_w;
        fj[i] = jj <= 2 * half_w ? (float)j : 3e9f;
        cj[i] = sgn * cospif((float)j / fhw);
        sj[i] = sgn * sinpif((float)j / fhw);
    }
    constexpr int NW = THREADS / 32;
    const unsigned h_addr = (unsigned)__cvta_generic_to_shared(h);
    // first-tap samples for which all 96 lane slots (81 of them taps) stay inside the response
    const unsigned inside = (unsigned)max(L - 96, 0);
    const bool mid_always = half_w >= 32;                       // taps 32..63 lie inside every window
    float4 *my4 = ring4 + warp * 32;
    float *my1 = ring1 + warp * 32;

    for (int base = warp * 32; base < total; base += NW * 32) {
        // ---- phase A: one image per lane
        const int idx = base + lane;
        bool valid = idx < total;
        float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
        float p2 = 0.f;
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
                int qq = idx - xpre[ix];              // position inside the diamond of radius r
                // rows ky = -r..0 hold 1, 3, .., 2r+1 points (qq < (r+1)^2, row u has u^2 before it);
                // rows ky = 1..r mirror rows r-1..0, counted from the end.
                const bool upper = qq >= (r + 1) * (r + 1);
                if (upper) qq = 2 * r * r + 2 * r - qq;
                int u = (int)sqrtf((float)qq);
                if (u * u > qq) --u;
                if ((u + 1) * (u + 1) <= qq) ++u;
                ky = upper ? r - u : u - r;
                kz = qq - u * u - u;
            }
            const int iy = ky + order, iz = kz + order;
            const double d2 = dsq[ix] + dsq[AX + iy] + dsq[2 * AX + iz];
            const float g = gain[ix] * gain[AX + iy] * gain[2 * AX + iz];
            // 1/d from the fp32 reciprocal square root and one Newton step in fp64
            // (relative error ~1e-14), d = d2/d with one correction
            double rd = (double)rsqrtf((float)d2);
            rd = fma(rd, 0.5 * fma(-d2 * rd, rd, 1.0), rd);
            double d = d2 * rd;
            d = fma(0.5 * rd, fma(-d, d, d2), d);
            const double tau = d * fs_over_c;
            const int n0 = __double2int_rn(tau);
            float phi = (float)(tau - (double)n0);
            // a fraction of exactly zero would make the centre tap 0/0: 1e-7 of a sample
            // away from it the tap is the same to 3e-7 of its size
            if (fabsf(phi) < 1e-7f) phi = copysignf(1e-7f, phi);
            const float A = g * (float)rd;
            valid = d2 > 0.0 && A != 0.f && n0 - half_w < L;
            const float As = -A * scale * sinpif(phi) * 0.318309886183790671538f;
            float sps, cps;
            sincospif(phi / fhw, &sps, &cps);
            q = make_float4(__int_as_float(n0), phi, 0.5f * As, 0.5f * As * cps);
            p2 = 0.5f * As * sps;
        }
        const unsigned mask = __ballot_sync(0xffffffffu, valid);
        if (valid) {
            const int pos = __popc(mask & ((1u << lane) - 1u));
            my4[pos] = q;
            my1[pos] = p2;
        }
        __syncwarp();
        // ---- phase B: the taps of one image over the lanes
        const int cnt = __popc(mask);
        for (int k = 0; k < cnt; ++k) {
            const float4 im = my4[k];
            const float P2 = my1[k];
            const int n_first = __float_as_int(im.x) - half_w;      // sample of tap -half_w
            const float phi = im.y, P0 = sgn * im.z, P1 = im.w;
            // A sinc(x) hann(x) = (1/x) (-A sin(pi phi)/pi) (-1)^j (1/2 + 1/2 cos(pi x / W_h)), x = j - phi
            if ((unsigned)n_first < inside) {
                // every tap of the window falls inside the response: no index checks, the
                // three adds go to fixed offsets from one address
                const unsigned a = h_addr + 4u * (unsigned)(n_first + lane);
                // (a predicated reduction compiles to a branch around it: a tap outside the
                // window adds zero instead; taps 32..63 are always inside it)
                const float x0 = fj[0] - phi, x1 = fj[1] - phi, x2 = fj[2] - phi;
                const float v0 = rcp_approx(x0) * fmaf(sj[0], P2, fmaf(cj[0], P1, P0));
                const float v1 = rcp_approx(x1) * fmaf(sj[1], P2, fmaf(cj[1], P1, P0));
                const float v2 = rcp_approx(x2) * fmaf(sj[2], P2, fmaf(cj[2], P1, P0));
                red_shared_add<0>(a, __float2int_rn(fabsf(x0) <= fhw ? v0 : 0.f));
                red_shared_add<128>(a, __float2int_rn(mid_always ? v1 : (fabsf(x1) <= fhw ? v1 : 0.f)));
                red_shared_add<256>(a, __float2int_rn(fabsf(x2) <= fhw ? v2 : 0.f));
            } else {
#pragma unroll
                for (int i = 0; i < 3; ++i) {
                    const float x = fj[i] - phi;
                    const int n = n_first + lane + 32 * i;
                    const float v = rcp_approx(x) * fmaf(sj[i], P2, fmaf(cj[i], P1, P0));
                    if (fabsf(x) <= fhw && (unsigned)n < (unsigned)L) atomicAdd(&h[n], __float2int_rn(v));
                }
            }
        }
        __syncwarp();   // the ring slots are rewritten by the next batch
    }
    __syncthreads();
    if ((reinterpret_cast<uintptr_t>(out) & 15) == 0 && (L & 3) == 0) {
        for (int i = tid; i < (L >> 2); i += THREADS) {
            const int4 q = reinterpret_cast<const int4 *>(h)[i];
            reinterpret_cast<float4 *>(out)[i] = make_float4((float)q.x * inv_scale, (float)q.y * inv_scale,
                                                             (float)q.z * inv_scale, (float)q.w * inv_scale);
        }
    } else {
        for (int i = tid; i < L; i += THREADS) out[i] = (float)h[i] * inv_scale;
    }
}

}  // namespace

int launch_rir(AugCtx *ctx, const AugUttParams *table, int B, float *rir, cudaStream_t st) {
    const AugConfig &c = ctx->cfg;
    const size_t smem = rir_smem_bytes(THREADS, c.rir_taps);
    const double fs_over_c = (double)c.fs / (double)c.sound_speed;
    const int cube = c.image_lattice == AUG_LATTICE_CUBE ? 1 : 0;
    dim3 grid(c.max_sources, B);
    if (smem_opt_in<rir_image_kernel>(ctx->device) != AUG_OK) return AUG_ECUDA;
    rir_image_kernel<<<grid, THREADS, smem, st>>>(table, c.max_sources, c.rir_taps, c.frac_half_width,
                                                  fs_over_c, c.max_order, cube, rir, ctx->status);
    AUG_CUDA_OK(cudaGetLastError());
    ctx->launches++;
    return AUG_OK;
}
