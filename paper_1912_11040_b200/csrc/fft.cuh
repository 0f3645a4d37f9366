// Shared-memory complex FFT building blocks (forward transform, e^{-i...}).
//
// A transform of N points is run by N/E threads; each pass keeps E points of a
// thread in registers as E/R radix-R butterflies and exchanges them through one
// shared-memory array in Stockham (self-sorting) order, so no bit reversal is
// needed.  The unnormalised inverse is obtained with the same code by swapping
// real and imaginary parts on the way in and on the way out.
#pragma once
#include <cuda_runtime.h>

namespace augfft {

// Twiddle table, TW_N entries: for every power of two M <= TW_N the block
// [M/2, M) holds exp(-2 pi i k / M), k < M/2, so that the factors one pass or one
// real-FFT split needs are contiguous in k (coalesced loads).
constexpr int TW_N = 16384;
__host__ __device__ constexpr int tw_index(int M, int k) { return M / 2 + k; }

__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cconj(float2 a) { return make_float2(a.x, -a.y); }
// a * (-i)
__device__ __forceinline__ float2 cmul_mi(float2 a) { return make_float2(a.y, -a.x); }

// In-register DFT of R points, natural order in and out.
template <int R>
struct Dft;

template <>
struct Dft<2> {
    __device__ __forceinline__ static void run(float2 *v) {
        float2 a = v[0], b = v[1];
        v[0] = cadd(a, b);
        v[1] = csub(a, b);
    }
};

template <>
struct Dft<4> {
    __device__ __forceinline__ static void run(float2 *v) {
        float2 t0 = cadd(v[0], v[2]), t1 = csub(v[0], v[2]);
        float2 t2 = cadd(v[1], v[3]), t3 = cmul_mi(csub(v[1], v[3]));
        v[0] = cadd(t0, t2);
        v[1] = cadd(t1, t3);
        v[2] = csub(t0, t2);
        v[3] = csub(t1, t3);
    }
};

template <>
struct Dft<8> {
    __device__ __forceinline__ static void run(float2 *v) {
        const float h = 0.70710678118654752440f;
        float2 e[4] = {v[0], v[2], v[4], v[6]};
        float2 o[4] = {v[1], v[3], v[5], v[7]};
        Dft<4>::run(e);
        Dft<4>::run(o);
        // o[k] *= exp(-2 pi i k / 8)
        o[1] = make_float2(h * (o[1].x + o[1].y), h * (o[1].y - o[1].x));
        o[2] = cmul_mi(o[2]);
        o[3] = make_float2(h * (o[3].y - o[3].x), -h * (o[3].x + o[3].y));
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            v[k] = cadd(e[k], o[k]);
            v[k + 4] = csub(e[k], o[k]);
        }
    }
};

template <>
struct Dft<16> {
    __device__ __forceinline__ static void run(float2 *v) {
        float2 e[8], o[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            e[k] = v[2 * k];
            o[k] = v[2 * k + 1];
        }
        Dft<8>::run(e);
        Dft<8>::run(o);
        const float c1 = 0.92387953251128675613f, s1 = 0.38268343236508977173f;
        const float h = 0.70710678118654752440f;
        // exp(-2 pi i k / 16), k = 1..7
        o[1] = cmul(o[1], make_float2(c1, -s1));
        o[2] = cmul(o[2], make_float2(h, -h));
        o[3] = cmul(o[3], make_float2(s1, -c1));
        o[4] = cmul_mi(o[4]);
        o[5] = cmul(o[5], make_float2(-s1, -c1));
        o[6] = cmul(o[6], make_float2(-h, -h));
        o[7] = cmul(o[7], make_float2(-c1, -s1));
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            v[k] = cadd(e[k], o[k]);
            v[k + 8] = csub(e[k], o[k]);
        }
    }
};

// Multiply v[r] by w^r, r = 1..R-1, with w = exp(-2 pi i k / (NS R)) read from the table.
// Powers are built by squaring (w^2, w^4, w^8) and one more product each, so no
// power is more than three roundings away from the table value.
template <int R>
__device__ __forceinline__ void twiddle_powers(float2 *w, float2 w1) {
    w[0] = make_float2(1.f, 0.f);
    w[1] = w1;
#pragma unroll
    for (int r = 2; r < R; ++r) {
        const int hi = (r & (r - 1)) ? (r & -r) : r / 2;   // split r = hi + lo with hi a power of two
        w[r] = cmul(w[hi], w[r - hi]);
    }
}
template <int R>
__device__ __forceinline__ void twiddle(float2 *v, float2 w1) {
    float2 w[R];
    twiddle_powers<R>(w, w1);
#pragma unroll
    for (int r = 1; r < R; ++r) v[r] = cmul(v[r], w[r]);
}

// Shared-memory index padding.  Complex points are 8 bytes, 16 of them span the 32
// banks.  Between passes element i lives at i + ((i >> 4) << PS), i.e. every row of
// 16 points is shifted by 1 (PS = 0) or 2 (PS = 1) slots per row.  Row-constant
// shifts keep the unit-stride gathers conflict-free; the shift is chosen per pass
// so that its scatter is conflict-free too: stride-R scatters (NS = 1) and the
// NS = 16 scatter want 1 per row, the NS = 8 scatter (rows 4 apart within a
// half-warp) wants 2 per row.  The last pass of a transform (NS >= 64 here) writes
// consecutive slots from consecutive threads and so do callers that fill a buffer
// themselves (NS = 0): those layouts are left unpadded (PS = -1), which also keeps
// mirrored reads (slot N-k next to slot k) free of conflicts.
template <int PS>
__device__ __forceinline__ int padi(int i) { return PS < 0 ? i : i + ((i >> 4) << (PS < 0 ? 0 : PS)); }
__host__ __device__ constexpr int padded_points(int n) { return n + n / 8; }
__host__ __device__ constexpr int out_shift(int NS) { return NS == 8 ? 1 : (NS == 1 || NS == 16) ? 0 : -1; }
// Index of point i in a finished transform or in a caller-written input: unpadded.
__device__ __forceinline__ int pad0(int i) { return i; }

// One pass over registers already holding the inputs of this thread's butterflies:
//   v[b][r] = data[(t + b T) + r N/R],  T = N/E threads, b < E/R.
// Applies the pass twiddles (NS = product of earlier radices), the radix-R DFTs,
// and scatters the results to `s` in Stockham order.  The caller synchronises.
// The same pass with the twiddle powers w[r] = w1^r of this thread's (single)
// butterfly already computed: two transforms that run the same pass side by side
// share them.
template <int N, int E, int R, int NS>
__device__ __forceinline__ void pass_from_regs_tw(float2 (*v)[R], float2 *s, int t, const float2 *w) {
    static_assert(E == R && NS > 1, "one butterfly per thread, a pass with twiddles");
    constexpr int PS = out_shift(NS);
    static_assert(PS >= 0 || NS * R == N, "only the last pass may write the unpadded layout");
    const int k = t & (NS - 1);
#pragma unroll
    for (int r = 1; r < R; ++r) v[0][r] = cmul(v[0][r], w[r]);
    Dft<R>::run(v[0]);
    const int base = padi<PS>((t - k) * R + k);
#pragma unroll
    for (int r = 0; r < R; ++r) s[base + padi<PS>(r * NS)] = v[0][r];
}

template <int N, int E, int R, int NS>
__device__ __forceinline__ void pass_from_regs(float2 (*v)[R], float2 *s, int t,
                                               const float2 *__restrict__ tw) {
    constexpr int T = N / E;
    constexpr int NB = E / R;
    constexpr int PS = out_shift(NS);
    static_assert(PS >= 0 || NS * R == N, "only the last pass may write the unpadded layout");
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        const int j = t + b * T;
        const int k = j & (NS - 1);
        if (NS > 1) {
            float2 w1 = __ldg(&tw[tw_index(NS * R, k)]);
            twiddle<R>(v[b], w1);
        }
        Dft<R>::run(v[b]);
        // Every r * NS is either a multiple of 16 or (NS = 8) stays inside j0's row
        // pair, so the padded address is padi(j0) plus a compile-time constant.
        const int base = padi<PS>((j - k) * R + k);
#pragma unroll
        for (int r = 0; r < R; ++r) s[base + padi<PS>(r * NS)] = v[b][r];
    }
}

// Gather the inputs of this thread's butterflies from `s`, laid out by the pass
// whose NS was NS_PREV (0 when the caller wrote the input with shift 0).
template <int N, int E, int R, int NS_PREV>
__device__ __forceinline__ void gather(float2 (*v)[R], const float2 *s, int t) {
    constexpr int T = N / E;
    constexpr int NB = E / R;
    constexpr int PS_IN = out_shift(NS_PREV);
    static_assert((N / R) % 16 == 0, "gather stride must keep the row offset constant");
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        const int base = padi<PS_IN>(t + b * T);
#pragma unroll
        for (int r = 0; r < R; ++r) v[b][r] = s[base + padi<PS_IN>(r * (N / R))];
    }
}

// A full pass: gather, barrier, transform, scatter, barrier.
template <int N, int E, int R, int NS, int NS_PREV, typename Sync>
__device__ __forceinline__ void pass(float2 *s, int t, const float2 *__restrict__ tw, Sync sync) {
    constexpr int NB = E / R;
    float2 v[NB][R];
    gather<N, E, R, NS_PREV>(v, s, t);
    sync();
    pass_from_regs<N, E, R, NS>(v, s, t, tw);
    sync();
}

// The same pass on two independent transforms in buffers `a` and `b`: the barrier
// that lets `a` be overwritten also publishes the previous writes to `b`, so the
// pair costs two barriers, not four.  On entry both buffers must be complete and
// visible; on exit `a` is complete and visible, `b` is written but not yet
// synchronised (the next pass_pair, or one barrier, finishes it).
template <int N, int E, int R, int NS, int NS_PREV, typename Sync>
__device__ __forceinline__ void pass_pair(float2 *a, float2 *b, int t, const float2 *__restrict__ tw,
                                          Sync sync) {
    constexpr int NB = E / R;
    float2 v[NB][R];
    if constexpr (NS > 1 && E == R) {
        // one butterfly per thread: both transforms use the same twiddle powers, built once
        float2 w[R];
        twiddle_powers<R>(w, __ldg(&tw[tw_index(NS * R, t & (NS - 1))]));
        // not unrolled: the second transform reuses the first one's instructions
        // (building the powers after the first gather instead, to hide the table load,
        // costs spills at this register budget and was slower)
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
            float2 *s = h ? b : a;
            gather<N, E, R, NS_PREV>(v, s, t);
            sync();
            pass_from_regs_tw<N, E, R, NS>(v, s, t, w);
        }
    } else {
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
            float2 *s = h ? b : a;
            gather<N, E, R, NS_PREV>(v, s, t);
            sync();
            pass_from_regs<N, E, R, NS>(v, s, t, tw);
        }
    }
}

struct CtaSync {
    __device__ __forceinline__ void operator()() const { __syncthreads(); }
};
// Barrier over `count` threads (whole warps) that share hardware barrier `id` (1..15).
struct GroupSync {
    int id, count;
    __device__ __forceinline__ void operator()() const {
        asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
    }
};

}  // namespace augfft
