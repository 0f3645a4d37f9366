// C ABI of libaugb200: argument checks, context and workspace, call sequencing.
#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>
#include <algorithm>
#include <vector>

#include "common.cuh"
#include "fft.cuh"

namespace {

inline int64_t align_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// Rows [b0, b1) of a padded batch in mapped pinned host memory -> the same rows of
// the device staging, each only up to its length (rounded up to whole groups of
// four samples, which the row stride always covers).  A small grid with many loads
// in flight per thread does best (48 x 256 threads x 16 loads; larger grids were
// slower), and the SMs stay free for the chunk that is being computed meanwhile.
// Neither this kernel nor the copy engine fills the host link alone with rows of this
// size (about 40 of 54 GB/s each), so a chunk's longest rows, AUG_DMA_SHARE_PCT percent
// of its samples, go by the copy engine at the same time on a stream of their own.
#ifndef AUG_DMA_SHARE_PCT
#define AUG_DMA_SHARE_PCT 40
#endif
#ifndef AUG_COPY_CTAS
#define AUG_COPY_CTAS 48
#endif
#ifndef AUG_COPY_UNROLL
#define AUG_COPY_UNROLL 16
#endif
constexpr int COPY_CTAS = AUG_COPY_CTAS, COPY_THREADS = 256, COPY_UNROLL = AUG_COPY_UNROLL;
#ifndef AUG_DMA_MIN_BYTES
#define AUG_DMA_MIN_BYTES (512 << 10)
#endif
constexpr int64_t DMA_MIN_BYTES = AUG_DMA_MIN_BYTES;   // feature blocks of this size go back by the copy engine
__global__ void __launch_bounds__(COPY_THREADS)
copy_rows_kernel(const float4 *__restrict__ src, float4 *__restrict__ dst, int64_t stride4,
                 const int *__restrict__ lengths, int b0, int b1, int below) {
    for (int b = b0; b < b1; ++b) {
        if (lengths[b] >= below) continue;      // that row travels by the copy engine
        const int n4 = (max(lengths[b], 0) + 3) >> 2;
        const float4 *s = src + (int64_t)b * stride4;
        float4 *d = dst + (int64_t)b * stride4;
        const int step = COPY_CTAS * COPY_THREADS;
        for (int i = blockIdx.x * COPY_THREADS + threadIdx.x; i < n4; i += step * COPY_UNROLL) {
            float4 v[COPY_UNROLL];
#pragma unroll
            for (int u = 0; u < COPY_UNROLL; ++u)
                if (i + u * step < n4) v[u] = s[i + u * step];
#pragma unroll
            for (int u = 0; u < COPY_UNROLL; ++u)
                if (i + u * step < n4) d[i + u * step] = v[u];
        }
    }
}

// The first counts[b] feature rows (row4 groups of four floats each) of utterances
// [b0, b1) from the device staging into the caller's mapped pinned buffer.
__global__ void __launch_bounds__(COPY_THREADS)
store_rows_kernel(const float4 *__restrict__ src, float4 *__restrict__ dst, int64_t utt4, int row4,
                  const int *__restrict__ counts, int b0, int b1, int below) {
    for (int b = b0; b < b1; ++b) {
        if (counts[b] >= below) continue;       // that utterance travels by the copy engine
        const int n4 = max(counts[b], 0) * row4;
        const float4 *s = src + (int64_t)b * utt4;
        float4 *d = dst + (int64_t)b * utt4;
        for (int i = blockIdx.x * COPY_THREADS + threadIdx.x; i < n4; i += COPY_CTAS * COPY_THREADS) d[i] = s[i];
    }
}

// Device-side alias of a host buffer if it is pinned and mapped, else NULL.
const float *mapped_alias(const float *host) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    if (a.type != cudaMemoryTypeHost || !a.devicePointer) return nullptr;
    return static_cast<const float *>(a.devicePointer);
}
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_config(const AugConfig *c) {
    if (!c) return AUG_EINVAL;
    if (c->fs <= 0 || c->hop <= 0 || c->win <= 0) return AUG_EINVAL;
    if (c->n_fft != 512 && c->n_fft != 1024) return AUG_EINVAL;
    if (c->win > c->n_fft) return AUG_EINVAL;
    if (c->n_mel < 1 || c->n_mel > aug::MAX_MEL) return AUG_EINVAL;
    if (!(c->f_lo >= 0.f) || !(c->f_hi > c->f_lo) || c->f_hi > 0.5f * c->fs + 1e-3f) return AUG_EINVAL;
    if (c->rir_taps < 1 || c->rir_taps > aug::MAX_TAPS) return AUG_EINVAL;
    if (c->max_order < 0 || c->max_order > aug::MAX_ORDER) return AUG_EINVAL;
    if (c->max_sources < 1 || c->max_sources > AUG_S_MAX) return AUG_EINVAL;
    if (c->frac_half_width < 1 || c->frac_half_width > aug::MAX_HALF_W) return AUG_EINVAL;
    if (!(c->sound_speed > 0.f) || !(c->log_floor > 0.f) || !isfinite(c->pad_value)) return AUG_EINVAL;
    if (c->compression != AUG_COMPRESS_LOG && c->compression != AUG_COMPRESS_POW_1_15) return AUG_EINVAL;
    if (c->image_lattice != AUG_LATTICE_TOTAL && c->image_lattice != AUG_LATTICE_CUBE) return AUG_EINVAL;
    if (c->host_rows != AUG_HOST_ROWS_PADDED && c->host_rows != AUG_HOST_ROWS_VALID) return AUG_EINVAL;
    if (c->max_batch < 1 || c->max_batch > 65535 || c->max_samples < 1) return AUG_EINVAL;
    if (c->host_staging && c->max_bank_samples < 0) return AUG_EINVAL;
    if (c->vtlp_win < 0 || c->vtlp_win > 1024 || (c->vtlp_win & 3)) return AUG_EINVAL;
    return AUG_OK;
}

struct Layout {
    int n_part, route, n_bins, t_cap, nblk_cap;
    int64_t ws_stride;
    int64_t off_xspec, off_park, off_park_flags;
    int64_t off_tw, off_rir, off_hspec, off_ys, off_vv, off_energy, off_leff, off_gain, off_melw, off_melstart,
        off_status, off_warped, off_vtlp_tab, off_st_speech, off_st_bank, off_st_table, off_st_lengths,
        off_st_feats, off_st_counts, total;
};

Layout make_layout(const AugConfig &c) {
    Layout l;
    l.n_part = (c.rir_taps + aug::CONV_BLK - 1) / aug::CONV_BLK;
    l.route = l.n_part <= 2 ? aug::ROUTE_FUSED_8192 : aug::ROUTE_STORED;
    l.n_bins = c.n_fft / 2 + 1;
    l.t_cap = aug_frame_count(c.max_samples, c.win, c.hop);
    l.ws_stride = align_up(c.max_samples, 4);
    const int64_t B = c.max_batch, S = c.max_sources;
    int64_t o = 0;
    auto take = [&](int64_t bytes) { int64_t r = o; o = align_up(o + bytes, 256); return r; };
    l.off_tw = take(sizeof(float2) * augfft::TW_N);
    l.off_rir = take(sizeof(float) * B * S * c.rir_taps);
    l.off_hspec = take(sizeof(float2) * B * S * (l.route == aug::ROUTE_FUSED_8192 ? 2 : l.n_part) * aug::CONV_N2);
    l.nblk_cap = (c.max_samples + aug::CONV_BLK - 1) / aug::CONV_BLK;
    l.off_xspec = l.route == aug::ROUTE_STORED ? take(sizeof(float2) * B * S * l.nblk_cap * aug::CONV_N2) : -1;
    // parking slots of the fused route, three per multiprocessor, when a row can have several noises
    const bool parks = c.max_sources >= 3;    // (long-response contexts use the fused route for short responses)
    l.off_park = parks ? take(sizeof(float2) * (int64_t)aug::PARK_SMS * aug::PARK_PER_SM * 2 * aug::CONV_N2) : -1;
    l.off_park_flags = parks ? take(sizeof(int) * (int64_t)aug::PARK_SMS * aug::PARK_PER_SM) : -1;
    l.off_ys = take(sizeof(float) * B * l.ws_stride);
    l.off_vv = take(sizeof(float) * B * l.ws_stride);
    l.off_energy = take(sizeof(double) * 2 * B);
    l.off_leff = take(sizeof(int) * (B + 1));
    l.off_gain = take(sizeof(float) * B);
    l.off_melw = take(sizeof(aug::MelBin) * B * l.n_bins);
    l.off_melstart = take(sizeof(int) * B * (c.n_mel + 2));
    l.off_status = take(sizeof(int) * 2);
    l.off_warped = c.vtlp_win > 0 ? take(sizeof(float) * B * l.ws_stride) : -1;
    l.off_vtlp_tab = c.vtlp_win > 0 ? take((sizeof(int) + sizeof(float)) * B * 513) : -1;
    if (c.host_staging) {
        l.off_st_speech = take(sizeof(float) * B * l.ws_stride);
        l.off_st_bank = take(sizeof(float) * (c.max_bank_samples > 0 ? c.max_bank_samples : 1));
        l.off_st_table = take(sizeof(AugUttParams) * B);
        l.off_st_lengths = take(sizeof(int) * B);
        l.off_st_feats = take(sizeof(float) * B * (int64_t)(l.t_cap > 0 ? l.t_cap : 1) * c.n_mel);
        l.off_st_counts = take(sizeof(int) * B);
    } else {
        l.off_st_speech = l.off_st_bank = l.off_st_table = l.off_st_lengths = l.off_st_feats =
            l.off_st_counts = -1;
    }
    l.total = o;
    return l;
}

// Common checks of the batch arguments; max_len_out = largest length if known from the host.
int check_batch(const AugCtx *ctx, int B) {
    if (!ctx) return AUG_EINVAL;
    if (B < 0) return AUG_EINVAL;
    if (B > ctx->cfg.max_batch) return AUG_ECAP;
    return AUG_OK;
}

}  // namespace

extern "C" {

const char *aug_strerror(int code) {
    switch (code) {
        case AUG_OK: return "success";
        case AUG_EINVAL: return "invalid argument (null or misaligned pointer, bad scalar)";
        case AUG_ECAP: return "request exceeds the capacity the context was created with";
        case AUG_ECUDA: return "CUDA runtime call or kernel launch failed";
        case AUG_EPARAM: return "parameter table row failed validation";
        case AUG_ENOMEM: return "device workspace allocation failed";
        default: return "unknown status code";
    }
}

int aug_frame_count(int n_samples, int win, int hop) {
    if (win <= 0 || hop <= 0 || n_samples < win) return 0;
    return 1 + (n_samples - win) / hop;
}

int64_t aug_workspace_bytes(const AugConfig *cfg) {
    int rc = check_config(cfg);
    if (rc != AUG_OK) return rc;
    return make_layout(*cfg).total;
}

int aug_validate_params(const AugConfig *cfg, const AugUttParams *tab, int B, int64_t bank_len,
                        int *bad_row) {
    if (bad_row) *bad_row = -1;
    if (!cfg || (!tab && B > 0) || B < 0) return AUG_EINVAL;
    for (int b = 0; b < B; ++b) {
        const AugUttParams &r = tab[b];
        bool ok = r.n_src >= 1 && r.n_src <= cfg->max_sources && r.order >= 0 &&
                  r.order <= cfg->max_order && isfinite(r.snr_db) && r.alpha > 0.f && r.alpha < 2.f;
        for (int a = 0; a < 3 && ok; ++a) {
            ok = isfinite(r.room[a]) && r.room[a] > 0.f && r.mic[a] >= 0.f && r.mic[a] <= r.room[a];
        }
        for (int w = 0; w < 6 && ok; ++w) ok = r.beta[w] >= 0.f && r.beta[w] <= 1.f;
        for (int s = 0; s < r.n_src && ok; ++s) {
            double d2 = 0.0;
            for (int a = 0; a < 3 && ok; ++a) {
                const float p = r.src_pos[s][a];
                ok = p >= 0.f && p <= r.room[a];
                d2 += ((double)p - r.mic[a]) * ((double)p - r.mic[a]);
            }
            if (ok) ok = d2 > 1e-12;   // a source on top of the microphone has no finite 1/d
        }
        for (int k = 0; k + 1 < r.n_src && ok; ++k) {
            ok = r.noise_len[k] > 0 && r.noise_offset[k] >= 0 &&
                 r.noise_offset[k] + r.noise_len[k] <= bank_len && isfinite(r.noise_weight[k]);
        }
        if (!ok) {
            if (bad_row) *bad_row = b;
            return AUG_EPARAM;
        }
    }
    return AUG_OK;
}

int aug_create(AugCtx **out, const AugConfig *cfg, void *cuda_stream) {
    if (!out) return AUG_EINVAL;
    *out = nullptr;
    int rc = check_config(cfg);
    if (rc != AUG_OK) return rc;
    AugCtx *ctx = new (std::nothrow) AugCtx();
    if (!ctx) return AUG_ENOMEM;
    memset(ctx, 0, sizeof(*ctx));
    ctx->cfg = *cfg;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaGetDevice(&ctx->device) != cudaSuccess) {
        delete ctx;
        return AUG_ECUDA;
    }
    if (cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&ctx->smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor,
                               ctx->device) != cudaSuccess) {
        delete ctx;
        return AUG_ECUDA;
    }
    const Layout l = make_layout(*cfg);
    ctx->n_part = l.n_part;
    ctx->route = l.route;
    ctx->n_bins = l.n_bins;
    ctx->t_cap = l.t_cap;
    ctx->ws_stride = l.ws_stride;
    ctx->ws_bytes = l.total;
    if (cudaMalloc(&ctx->ws_base, (size_t)l.total) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return AUG_ENOMEM;
    }
    char *base = static_cast<char *>(ctx->ws_base);
    ctx->tw = reinterpret_cast<float2 *>(base + l.off_tw);
    ctx->rir = reinterpret_cast<float *>(base + l.off_rir);
    ctx->hspec = reinterpret_cast<float2 *>(base + l.off_hspec);
    ctx->nblk_cap = l.nblk_cap;
    ctx->xspec = l.off_xspec >= 0 ? reinterpret_cast<float2 *>(base + l.off_xspec) : nullptr;
    ctx->park = l.off_park >= 0 ? reinterpret_cast<float2 *>(base + l.off_park) : nullptr;
    ctx->park_flags = l.off_park_flags >= 0 ? reinterpret_cast<int *>(base + l.off_park_flags) : nullptr;
    ctx->n_sm = aug::PARK_SMS;
    ctx->ys = reinterpret_cast<float *>(base + l.off_ys);
    ctx->vv = reinterpret_cast<float *>(base + l.off_vv);
    ctx->energy = reinterpret_cast<double *>(base + l.off_energy);
    ctx->leff = reinterpret_cast<int *>(base + l.off_leff);
    ctx->gain = reinterpret_cast<float *>(base + l.off_gain);
    ctx->melw = reinterpret_cast<aug::MelBin *>(base + l.off_melw);
    ctx->melstart = reinterpret_cast<int *>(base + l.off_melstart);
    ctx->status = reinterpret_cast<int *>(base + l.off_status);
    ctx->warped = l.off_warped >= 0 ? reinterpret_cast<float *>(base + l.off_warped) : nullptr;
    ctx->vtlp_tab = l.off_vtlp_tab >= 0 ? base + l.off_vtlp_tab : nullptr;
    if (cfg->host_staging) {
        ctx->st_speech = reinterpret_cast<float *>(base + l.off_st_speech);
        ctx->st_bank = reinterpret_cast<float *>(base + l.off_st_bank);
        ctx->st_table = reinterpret_cast<AugUttParams *>(base + l.off_st_table);
        ctx->st_lengths = reinterpret_cast<int *>(base + l.off_st_lengths);
        ctx->st_feats = reinterpret_cast<float *>(base + l.off_st_feats);
        ctx->st_counts = reinterpret_cast<int *>(base + l.off_st_counts);
    }
    if (ctx->route == aug::ROUTE_STORED) {
        if (cudaHostAlloc(reinterpret_cast<void **>(&ctx->leff_seen), sizeof(int), cudaHostAllocDefault) !=
            cudaSuccess) {
            cudaGetLastError();
            cudaFree(ctx->ws_base);
            delete ctx;
            return AUG_ENOMEM;
        }
        *ctx->leff_seen = 0;
    }
    // The filterbank tables depend on the parameter table alone: aug_pipeline builds them on a
    // stream of their own while the impulse responses are computed (without it, in line).
    if (cudaStreamCreateWithFlags(&ctx->s_side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
        if (ctx->s_side) cudaStreamDestroy(ctx->s_side);
        ctx->s_side = nullptr;
        ctx->ev_fork = ctx->ev_join = nullptr;
    }
    if (cfg->host_staging) {
        bool ok_s = cudaStreamCreateWithFlags(&ctx->s_h2d, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaStreamCreateWithFlags(&ctx->s_h2d2, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaEventCreateWithFlags(&ctx->ev_len, cudaEventDisableTiming) == cudaSuccess &&
                    cudaStreamCreateWithFlags(&ctx->s_d2h, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < aug::HOST_CHUNKS && ok_s; ++i)
            ok_s = cudaEventCreateWithFlags(&ctx->ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
                   cudaEventCreateWithFlags(&ctx->ev_in2[i], cudaEventDisableTiming) == cudaSuccess &&
                   cudaEventCreateWithFlags(&ctx->ev_out[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok_s) {
            if (ctx->leff_seen) cudaFreeHost(ctx->leff_seen);
            cudaFree(ctx->ws_base);
            delete ctx;
            return AUG_ECUDA;
        }
    }
    // twiddles, evaluated in double: block [M/2, M) = exp(-2 pi i k / M), k < M/2
    std::vector<float2> tw(augfft::TW_N);
    tw[0] = make_float2(1.f, 0.f);
    for (int M = 2; M <= augfft::TW_N; M *= 2) {
        for (int k = 0; k < M / 2; ++k) {
            const double a = -2.0 * 3.14159265358979323846 * k / M;
            tw[augfft::tw_index(M, k)] = make_float2((float)cos(a), (float)sin(a));
        }
    }
    const int st0[2] = {-1, 0};
    if (ctx->park_flags &&
        cudaMemsetAsync(ctx->park_flags, 0, sizeof(int) * aug::PARK_SMS * aug::PARK_PER_SM, ctx->stream) !=
            cudaSuccess) {
        if (ctx->leff_seen) cudaFreeHost(ctx->leff_seen);
        cudaFree(ctx->ws_base);
        delete ctx;
        return AUG_ECUDA;
    }
    bool ok = cudaMemcpyAsync(ctx->tw, tw.data(), sizeof(float2) * augfft::TW_N,
                              cudaMemcpyHostToDevice, ctx->stream) == cudaSuccess &&
              cudaMemcpyAsync(ctx->status, st0, sizeof(st0), cudaMemcpyHostToDevice,
                              ctx->stream) == cudaSuccess &&
              cudaStreamSynchronize(ctx->stream) == cudaSuccess;
    if (!ok) {
        if (ctx->leff_seen) cudaFreeHost(ctx->leff_seen);
        cudaFree(ctx->ws_base);
        delete ctx;
        return AUG_ECUDA;
    }
    *out = ctx;
    return AUG_OK;
}

int aug_destroy(AugCtx *ctx) {
    if (!ctx) return AUG_OK;
    int rc = AUG_OK;
    if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) rc = AUG_ECUDA;
    if (ctx->ev) {
        for (int i = 0; i < aug::EV_RING * 2 * AUG_N_STAGES; ++i) cudaEventDestroy(ctx->ev[i]);
        free(ctx->ev);
    }

    if (ctx->s_side) {
        cudaStreamSynchronize(ctx->s_side);
        cudaEventDestroy(ctx->ev_fork);
        cudaEventDestroy(ctx->ev_join);
        cudaStreamDestroy(ctx->s_side);
    }
    if (ctx->s_h2d) {
        cudaStreamSynchronize(ctx->s_h2d);
        cudaStreamSynchronize(ctx->s_d2h);
        if (ctx->s_h2d2) {
            cudaStreamSynchronize(ctx->s_h2d2);
            cudaStreamDestroy(ctx->s_h2d2);
        }
        if (ctx->ev_len) cudaEventDestroy(ctx->ev_len);
        for (int i = 0; i < aug::HOST_CHUNKS; ++i) {
            if (ctx->ev_in2[i]) cudaEventDestroy(ctx->ev_in2[i]);
            cudaEventDestroy(ctx->ev_in[i]);
            cudaEventDestroy(ctx->ev_out[i]);
        }
        cudaEventDestroy(ctx->ev_start);
        cudaStreamDestroy(ctx->s_h2d);
        cudaStreamDestroy(ctx->s_d2h);
    }
    if (ctx->leff_seen) cudaFreeHost(ctx->leff_seen);
    if (cudaFree(ctx->ws_base) != cudaSuccess) rc = AUG_ECUDA;
    delete ctx;
    return rc;
}

int aug_last_status(AugCtx *ctx, int *utt, int *reason) {
    if (!ctx) return AUG_EINVAL;
    int st[2] = {-1, 0};
    AUG_CUDA_OK(cudaMemcpyAsync(st, ctx->status, sizeof(st), cudaMemcpyDeviceToHost, ctx->stream));
    AUG_CUDA_OK(cudaStreamSynchronize(ctx->stream));
    const int clear[2] = {-1, 0};
    AUG_CUDA_OK(cudaMemcpyAsync(ctx->status, clear, sizeof(clear), cudaMemcpyHostToDevice, ctx->stream));
    AUG_CUDA_OK(cudaStreamSynchronize(ctx->stream));
    if (utt) *utt = st[0];
    if (reason) *reason = st[0] >= 0 ? st[1] : 0;
    return AUG_OK;
}

int aug_vtlp_resynth(AugCtx *ctx, const float *speech_dev, int64_t stride, const int *lengths_dev,
                     const AugUttParams *table_dev, int B, float *warped_dev, int64_t out_stride) {
    int rc = check_batch(ctx, B);
    if (rc != AUG_OK) return rc;
    if (ctx->cfg.vtlp_win <= 0) return AUG_EINVAL;
    if (B == 0) return AUG_OK;
    if (!speech_dev || !lengths_dev || !table_dev || !warped_dev || stride <= 0 || out_stride <= 0)
        return AUG_EINVAL;
    const int64_t cap = stride < out_stride ? stride : out_stride;
    const int max_len = (int)(cap < ctx->cfg.max_samples ? cap : ctx->cfg.max_samples);
    return launch_vtlp_resynth(ctx, speech_dev, stride, lengths_dev, table_dev, B, max_len, warped_dev,
                               out_stride);
}

int aug_rir_image_method(AugCtx *ctx, const AugUttParams *table_dev, int B, float *rir_dev) {
    int rc = check_batch(ctx, B);
    if (rc != AUG_OK) return rc;
    if (B == 0) return AUG_OK;
    if (!table_dev || !rir_dev || !aligned16(rir_dev)) return AUG_EINVAL;
    return launch_rir(ctx, table_dev, B, rir_dev, ctx->stream);
}

int aug_reverb_mix(AugCtx *ctx, const float *speech_dev, int64_t speech_stride,
                   const int *lengths_dev, const float *noise_bank_dev, int64_t bank_len,
                   const float *rir_dev, const AugUttParams *table_dev, int B, float *wave_out_dev) {
    int rc = check_batch(ctx, B);
    if (rc != AUG_OK) return rc;
    if (B == 0) return AUG_OK;
    if (!speech_dev || !lengths_dev || !rir_dev || !table_dev || !wave_out_dev) return AUG_EINVAL;
    if (!aligned16(speech_dev) || !aligned16(wave_out_dev) || !aligned16(rir_dev)) return AUG_EINVAL;
    if (noise_bank_dev && !aligned16(noise_bank_dev)) return AUG_EINVAL;
    if (speech_stride <= 0 || (speech_stride & 3) || bank_len < 0) return AUG_EINVAL;
    const int max_len = (int)(speech_stride < ctx->cfg.max_samples ? speech_stride : ctx->cfg.max_samples);
    if (speech_stride > ctx->ws_stride) return AUG_ECAP;
    if ((rc = launch_rir_spectra(ctx, rir_dev, table_dev, B, ctx->stream)) != AUG_OK) return rc;
    if ((rc = launch_convolve_prepare(ctx, speech_dev, speech_stride, lengths_dev, noise_bank_dev,
                                      bank_len, table_dev, B, max_len)) != AUG_OK) return rc;
    if ((rc = launch_convolve_finish(ctx, speech_dev, speech_stride, lengths_dev, noise_bank_dev,
                                     bank_len, table_dev, B, max_len)) != AUG_OK) return rc;
    return launch_mix(ctx, lengths_dev, table_dev, B, max_len, wave_out_dev, speech_stride);
}

int feat_stft_power(AugCtx *ctx, const float *wave_dev, int64_t stride, const int *lengths_dev,
                    int B, float *power_dev, int T_max, int *frame_counts_dev) {
    int rc = check_batch(ctx, B);
    if (rc != AUG_OK) return rc;
    if (B == 0) return AUG_OK;
    if (!wave_dev || !lengths_dev || !power_dev || !frame_counts_dev) return AUG_EINVAL;
    if (!aligned16(wave_dev) || stride <= 0 || T_max < 0) return AUG_EINVAL;
    if (T_max == 0) return AUG_EINVAL;
    return launch_stft_power(ctx, wave_dev, stride, lengths_dev, B, power_dev, T_max, frame_counts_dev);
}

int feat_vtlp_logmel(AugCtx *ctx, const float *power_dev, const int *frame_counts_dev,
                     const AugUttParams *table_dev, int B, int T_max, float *feats_dev) {
    int rc = check_batch(ctx, B);
    if (rc != AUG_OK) return rc;
    if (B == 0) return AUG_OK;
    if (!power_dev || !frame_counts_dev || !table_dev || !feats_dev || T_max <= 0) return AUG_EINVAL;
    if ((rc = launch_mel_tables(ctx, table_dev, B, ctx->stream)) != AUG_OK) return rc;
    return launch_logmel(ctx, power_dev, frame_counts_dev, B, T_max, feats_dev);
}

int aug_pipeline(AugCtx *ctx, const float *speech_dev, int64_t speech_stride,
                 const int *lengths_dev, const int *lengths_host, const float *noise_bank_dev,
                 int64_t bank_len, const AugUttParams *table_dev, int B, float *feats_dev,
                 int T_max, int *frame_counts_dev, float *wave_out) {
    int rc = check_batch(ctx, B);
    if (rc != AUG_OK) return rc;
    if (B == 0) return AUG_OK;
    if (!speech_dev || !lengths_dev || !table_dev || !feats_dev || !frame_counts_dev) return AUG_EINVAL;
    if (!aligned16(speech_dev) || !aligned16(feats_dev)) return AUG_EINVAL;
    if (noise_bank_dev && !aligned16(noise_bank_dev)) return AUG_EINVAL;
    if (wave_out && !aligned16(wave_out)) return AUG_EINVAL;
    if (speech_stride <= 0 || (speech_stride & 3) || bank_len < 0 || T_max <= 0) return AUG_EINVAL;
    if (speech_stride > ctx->ws_stride) return AUG_ECAP;
    int max_len = (int)(speech_stride < ctx->cfg.max_samples ? speech_stride : ctx->cfg.max_samples);
    if (lengths_host) {
        int mx = 0;
        for (int b = 0; b < B; ++b) {
            if (lengths_host[b] < 0) return AUG_EINVAL;
            if (lengths_host[b] > max_len) return AUG_ECAP;
            if (lengths_host[b] > mx) mx = lengths_host[b];
        }
        if (aug_frame_count(mx, ctx->cfg.win, ctx->cfg.hop) > T_max) return AUG_ECAP;
        max_len = mx;
    }
    // Stage timing: a start and a stop event per stage, on the stream the stage runs on.
    cudaEvent_t *ev = nullptr;
    if (ctx->timing && ctx->ev && ctx->ev_n < aug::EV_RING)
        ev = ctx->ev + (size_t)ctx->ev_n * (2 * AUG_N_STAGES);
    auto t0 = [&](int stage, cudaStream_t st) { if (ev) cudaEventRecord(ev[2 * stage], st); };
    auto t1 = [&](int stage, cudaStream_t st) { if (ev) cudaEventRecord(ev[2 * stage + 1], st); };
    // Running the impulse-response chain beside the block spectra on a second stream was
    // measured and gained nothing (both saturate the SMs' issue and shared-memory pipes), so
    // those stages follow one another.  Only the small filterbank-table kernel, which needs
    // nothing but the parameter table, runs beside them on the side stream.
    cudaStream_t sm = ctx->stream, ss = ctx->stream;
    cudaStream_t st_mel = ctx->s_side ? ctx->s_side : ss;
    if (ctx->s_side) {
        AUG_CUDA_OK(cudaEventRecord(ctx->ev_fork, ss));     // after the caller's earlier work, this context's too
        AUG_CUDA_OK(cudaStreamWaitEvent(ctx->s_side, ctx->ev_fork, 0));
        t0(2, st_mel);
        rc = launch_mel_tables(ctx, table_dev, B, st_mel);
        t1(2, st_mel);
        if (rc != AUG_OK) return rc;
        AUG_CUDA_OK(cudaEventRecord(ctx->ev_join, ctx->s_side));
    }
    // every way out from here on first lets the context's stream wait for the side stream
    auto joined = [&](int code) {
        if (ctx->s_side && cudaStreamWaitEvent(sm, ctx->ev_join, 0) != cudaSuccess && code == AUG_OK)
            return (int)AUG_ECUDA;
        return code;
    };
    t0(0, ss);
    rc = launch_rir(ctx, table_dev, B, ctx->rir, ss);
    t1(0, ss);
    t0(1, ss);
    if (rc == AUG_OK) rc = launch_rir_spectra(ctx, ctx->rir, table_dev, B, ss);
    t1(1, ss);
    if (!ctx->s_side) {
        t0(2, ss);
        if (rc == AUG_OK) rc = launch_mel_tables(ctx, table_dev, B, ss);
        t1(2, ss);
    }

    // waveform-domain warp first: the simulator then sees the warped speech (timed with stage 3)
    t0(3, sm);
    if (rc == AUG_OK && ctx->warped) {
        rc = launch_vtlp_resynth(ctx, speech_dev, speech_stride, lengths_dev, table_dev, B, max_len,
                                 ctx->warped, ctx->ws_stride);
        speech_dev = ctx->warped;
        speech_stride = ctx->ws_stride;
    }
    if (rc == AUG_OK)
        rc = launch_convolve_prepare(ctx, speech_dev, speech_stride, lengths_dev, noise_bank_dev,
                                     bank_len, table_dev, B, max_len);
    t1(3, sm);
    if (rc != AUG_OK) return joined(rc);
    t0(4, sm);
    rc = launch_convolve_finish(ctx, speech_dev, speech_stride, lengths_dev, noise_bank_dev, bank_len,
                                table_dev, B, max_len);
    t1(4, sm);
    if (rc != AUG_OK) return joined(rc);
    t0(5, sm);
    if (wave_out &&
        (rc = launch_mix(ctx, lengths_dev, table_dev, B, max_len, wave_out, speech_stride)) != AUG_OK)
        return joined(rc);
    t1(5, sm);
    if ((rc = joined(AUG_OK)) != AUG_OK) return rc;
    t0(6, sm);
    rc = launch_fused_features(ctx, lengths_dev, table_dev, B, feats_dev, T_max, frame_counts_dev, max_len);
    t1(6, sm);
    if (ev && rc == AUG_OK) ctx->ev_n++;
    return rc;
}

int aug_pipeline_host(AugCtx *ctx, const float *speech_host, int64_t speech_stride,
                      const int *lengths_host, const float *noise_bank_host, int64_t bank_len,
                      const AugUttParams *table_host, int B, float *feats_host, int T_max,
                      int *frame_counts_host) {
    int rc = check_batch(ctx, B);
    if (rc != AUG_OK) return rc;
    if (!ctx->st_speech) return AUG_EINVAL;   // context created without host_staging
    if (B == 0) return AUG_OK;
    if (!speech_host || !lengths_host || !table_host || !feats_host || !frame_counts_host) return AUG_EINVAL;
    if (speech_stride <= 0 || (speech_stride & 3) || bank_len < 0 || T_max <= 0) return AUG_EINVAL;
    if (speech_stride > ctx->ws_stride || bank_len > ctx->cfg.max_bank_samples || T_max > ctx->t_cap)
        return AUG_ECAP;
    // no bank pointer: the bank uploaded earlier with aug_upload_noise_bank, of this length
    if (bank_len > 0 && !noise_bank_host && ctx->bank_resident != bank_len) return AUG_EINVAL;
    for (int b = 0; b < B; ++b)
        if (lengths_host[b] < 0 || lengths_host[b] > speech_stride) return AUG_EINVAL;

    // Software pipeline over chunks of utterances: chunk c+1 is copied in while chunk
    // c is computed and chunk c-1 is copied out, on three streams tied by events.
    // Rows are copied only up to their length when the bytes saved outweigh the
    // cost of one copy call per row.
    cudaStream_t sc = ctx->stream, si = ctx->s_h2d, si2 = ctx->s_h2d2, so = ctx->s_d2h;
    int64_t total = 0;
    for (int b = 0; b < B; ++b) total += lengths_host[b];
    const double saved_s = (double)((int64_t)B * speech_stride - total) * sizeof(float) / 40e9;
    const bool ragged = saved_s > (double)B * 4e-6;
    // Ragged rows of a pinned, mapped buffer are fetched by a small kernel that reads
    // host memory directly: one launch per chunk instead of one copy per row (copies
    // of a few hundred kilobytes each reach about 70 % of the link's rate).
    const float *speech_alias = ragged && (reinterpret_cast<uintptr_t>(speech_host) & 15) == 0
                                    ? mapped_alias(speech_host) : nullptr;
    const int n_chunk = B >= 2 * aug::HOST_CHUNKS ? aug::HOST_CHUNKS : 1;

    AUG_CUDA_OK(cudaEventRecord(ctx->ev_start, sc));          // earlier work on the context's stream
    AUG_CUDA_OK(cudaStreamWaitEvent(si, ctx->ev_start, 0));
    AUG_CUDA_OK(cudaMemcpyAsync(ctx->st_table, table_host, sizeof(AugUttParams) * (size_t)B,
                                cudaMemcpyHostToDevice, si));
    AUG_CUDA_OK(cudaMemcpyAsync(ctx->st_lengths, lengths_host, sizeof(int) * (size_t)B,
                                cudaMemcpyHostToDevice, si));
    if (speech_alias) {
        // the gather kernel's stream starts once the lengths are on the device
        AUG_CUDA_OK(cudaEventRecord(ctx->ev_len, si));
        AUG_CUDA_OK(cudaStreamWaitEvent(si2, ctx->ev_len, 0));
    }
    if (bank_len > 0 && noise_bank_host) {
        AUG_CUDA_OK(cudaMemcpyAsync(ctx->st_bank, noise_bank_host, sizeof(float) * (size_t)bank_len,
                                    cudaMemcpyHostToDevice, si));
        ctx->bank_resident = 0;   // the staging copy now holds this call's bank
    }
    const int M = ctx->cfg.n_mel;
    ctx->last_h2d = (int64_t)sizeof(AugUttParams) * B + (int64_t)sizeof(int) * B +
                    (int64_t)sizeof(float) * (noise_bank_host ? bank_len : 0) +
                    (int64_t)sizeof(float) * (ragged ? total : (int64_t)B * speech_stride);
    const bool valid_rows = ctx->cfg.host_rows == AUG_HOST_ROWS_VALID;
    // frames per utterance as the device will count them (lengths are cut at the row stride)
    auto frames_of = [&](int b) {
        return std::min(aug_frame_count((int)std::min<int64_t>(lengths_host[b], speech_stride), ctx->cfg.win,
                                        ctx->cfg.hop), T_max);
    };
    int64_t rows_out = (int64_t)B * T_max;
    if (valid_rows) {
        rows_out = 0;
        for (int b = 0; b < B; ++b) rows_out += frames_of(b);
    }
    ctx->last_d2h = (int64_t)sizeof(float) * rows_out * M + (int64_t)sizeof(int) * B;
    float *feats_alias = nullptr;
    if (valid_rows && (M & 3) == 0 && aligned16(feats_host))
        feats_alias = const_cast<float *>(mapped_alias(feats_host));
    int b0 = 0;
    int64_t done = 0;
    for (int c = 0; c < n_chunk; ++c) {
        // chunk boundaries at equal shares of the samples
        int b1 = b0;
        const int64_t goal = total * (c + 1) / n_chunk;
        while (b1 < B && (done < goal || b1 == b0)) done += lengths_host[b1++];
        if (c == n_chunk - 1) b1 = B;
        if (b1 == b0) continue;
        const int nb = b1 - b0;
        if (speech_alias) {
            // rows of at least `below` samples by the copy engine (the longest rows, up to its
            // share of the chunk's samples), the others by the kernel, both at once
            int below = 0x7fffffff;
            if (AUG_DMA_SHARE_PCT > 0 && nb > 1) {
                std::vector<int> len(lengths_host + b0, lengths_host + b1);
                std::sort(len.begin(), len.end(), [](int a, int b) { return a > b; });
                int64_t chunk_total = 0, acc = 0;
                for (int v : len) chunk_total += v;
                for (int v : len) {
                    if ((acc + v) * 100 > chunk_total * AUG_DMA_SHARE_PCT) break;
                    acc += v;
                    below = v;
                }
            }
            for (int b = b0; b < b1; ++b)
                if (lengths_host[b] >= below)
                    AUG_CUDA_OK(cudaMemcpyAsync(ctx->st_speech + (int64_t)b * speech_stride,
                                                speech_host + (int64_t)b * speech_stride,
                                                sizeof(float) * (size_t)lengths_host[b],
                                                cudaMemcpyHostToDevice, si));
            copy_rows_kernel<<<COPY_CTAS, COPY_THREADS, 0, si2>>>(
                reinterpret_cast<const float4 *>(speech_alias), reinterpret_cast<float4 *>(ctx->st_speech),
                speech_stride / 4, ctx->st_lengths, b0, b1, below);
            AUG_CUDA_OK(cudaGetLastError());
            ctx->launches++;
            AUG_CUDA_OK(cudaEventRecord(ctx->ev_in2[c], si2));
            AUG_CUDA_OK(cudaStreamWaitEvent(sc, ctx->ev_in2[c], 0));
        } else if (ragged) {
            for (int b = b0; b < b1; ++b)
                if (lengths_host[b] > 0)
                    AUG_CUDA_OK(cudaMemcpyAsync(ctx->st_speech + (int64_t)b * speech_stride,
                                                speech_host + (int64_t)b * speech_stride,
                                                sizeof(float) * (size_t)lengths_host[b],
                                                cudaMemcpyHostToDevice, si));
        } else {
            AUG_CUDA_OK(cudaMemcpyAsync(ctx->st_speech + (int64_t)b0 * speech_stride,
                                        speech_host + (int64_t)b0 * speech_stride,
                                        sizeof(float) * (size_t)nb * speech_stride,
                                        cudaMemcpyHostToDevice, si));
        }
        AUG_CUDA_OK(cudaEventRecord(ctx->ev_in[c], si));
        AUG_CUDA_OK(cudaStreamWaitEvent(sc, ctx->ev_in[c], 0));
        float *f_dev = ctx->st_feats + (int64_t)b0 * T_max * M;
        rc = aug_pipeline(ctx, ctx->st_speech + (int64_t)b0 * speech_stride, speech_stride,
                          ctx->st_lengths + b0, lengths_host + b0,
                          bank_len > 0 ? ctx->st_bank : nullptr, bank_len, ctx->st_table + b0, nb,
                          f_dev, T_max, ctx->st_counts + b0, nullptr);
        if (rc != AUG_OK) break;
        AUG_CUDA_OK(cudaEventRecord(ctx->ev_out[c], sc));
        AUG_CUDA_OK(cudaStreamWaitEvent(so, ctx->ev_out[c], 0));
        if (feats_alias) {
            // utterances with at least DMA_MIN_BYTES of features by the copy engine (it moves
            // large blocks faster than stores from a kernel do), the others by the kernel
            const int below = (int)std::min<int64_t>(0x7fffffff, (DMA_MIN_BYTES + 4 * M - 1) / (4 * M));
            bool any_small = false;
            for (int b = b0; b < b1; ++b) {
                const int T = frames_of(b);
                if (T >= below) {
                    // utterances that fill all T_max rows run on into the next one: one copy
                    int64_t rows = T;
                    const int first = b;
                    while (frames_of(b) == T_max && b + 1 < b1 && frames_of(b + 1) >= below)
                        rows = (int64_t)(++b - first) * T_max + frames_of(b);
                    AUG_CUDA_OK(cudaMemcpyAsync(feats_host + (int64_t)first * T_max * M,
                                                ctx->st_feats + (int64_t)first * T_max * M,
                                                sizeof(float) * (size_t)rows * M, cudaMemcpyDeviceToHost, so));
                } else if (T > 0) {
                    any_small = true;
                }
            }
            if (any_small) {
                store_rows_kernel<<<COPY_CTAS, COPY_THREADS, 0, so>>>(
                    reinterpret_cast<const float4 *>(ctx->st_feats), reinterpret_cast<float4 *>(feats_alias),
                    (int64_t)T_max * M / 4, M / 4, ctx->st_counts, b0, b1, below);
                AUG_CUDA_OK(cudaGetLastError());
                ctx->launches++;
            }
        } else if (valid_rows) {
            for (int b = b0; b < b1; ++b)
                if (frames_of(b) > 0)
                    AUG_CUDA_OK(cudaMemcpyAsync(feats_host + (int64_t)b * T_max * M,
                                                ctx->st_feats + (int64_t)b * T_max * M,
                                                sizeof(float) * (size_t)frames_of(b) * M,
                                                cudaMemcpyDeviceToHost, so));
        } else {
            AUG_CUDA_OK(cudaMemcpyAsync(feats_host + (int64_t)b0 * T_max * M, f_dev,
                                        sizeof(float) * (size_t)nb * T_max * M, cudaMemcpyDeviceToHost, so));
        }
        AUG_CUDA_OK(cudaMemcpyAsync(frame_counts_host + b0, ctx->st_counts + b0, sizeof(int) * (size_t)nb,
                                    cudaMemcpyDeviceToHost, so));
        b0 = b1;
    }
    // drain all three streams whatever happened above
    const bool ok = cudaStreamSynchronize(si) == cudaSuccess && cudaStreamSynchronize(si2) == cudaSuccess &&
                    cudaStreamSynchronize(sc) == cudaSuccess &&
                    cudaStreamSynchronize(so) == cudaSuccess;
    if (rc != AUG_OK) return rc;
    return ok ? AUG_OK : AUG_ECUDA;
}

int aug_upload_noise_bank(AugCtx *ctx, const float *noise_bank_host, int64_t bank_len) {
    if (!ctx || !noise_bank_host || bank_len <= 0) return AUG_EINVAL;
    if (!ctx->st_bank) return AUG_EINVAL;   // context created without host_staging
    if (bank_len > ctx->cfg.max_bank_samples) return AUG_ECAP;
    ctx->bank_resident = 0;
    AUG_CUDA_OK(cudaMemcpyAsync(ctx->st_bank, noise_bank_host, sizeof(float) * (size_t)bank_len,
                                cudaMemcpyHostToDevice, ctx->stream));
    AUG_CUDA_OK(cudaStreamSynchronize(ctx->stream));
    ctx->bank_resident = bank_len;
    return AUG_OK;
}

int aug_hold_parking_slots(AugCtx *ctx, int hold) {
    if (!ctx) return AUG_EINVAL;
    if (!ctx->park_flags) return AUG_OK;   // this context has no parking area
    // all slots marked taken: every CTA then sums its noise sources in the time domain
    std::vector<int> v((size_t)aug::PARK_SMS * aug::PARK_PER_SM, hold ? 1 : 0);
    AUG_CUDA_OK(cudaStreamSynchronize(ctx->stream));
    AUG_CUDA_OK(cudaMemcpyAsync(ctx->park_flags, v.data(), sizeof(int) * v.size(), cudaMemcpyHostToDevice,
                                ctx->stream));
    AUG_CUDA_OK(cudaStreamSynchronize(ctx->stream));
    return AUG_OK;
}

int aug_enable_stage_timing(AugCtx *ctx, int on) {
    if (!ctx) return AUG_EINVAL;
    AUG_CUDA_OK(cudaStreamSynchronize(ctx->stream));
    if (on && !ctx->ev) {
        const int n = aug::EV_RING * 2 * AUG_N_STAGES;
        ctx->ev = static_cast<cudaEvent_t *>(calloc(n, sizeof(cudaEvent_t)));
        if (!ctx->ev) return AUG_ENOMEM;
        for (int i = 0; i < n; ++i) {
            if (cudaEventCreate(&ctx->ev[i]) != cudaSuccess) {
                for (int j = 0; j < i; ++j) cudaEventDestroy(ctx->ev[j]);
                free(ctx->ev);
                ctx->ev = nullptr;
                return AUG_ECUDA;
            }
        }
    }
    ctx->timing = on ? 1 : 0;
    ctx->ev_n = 0;
    return AUG_OK;
}

int aug_stage_times(AugCtx *ctx, float *ms_host, int *n_calls_host) {
    if (!ctx || !ms_host) return AUG_EINVAL;
    AUG_CUDA_OK(cudaStreamSynchronize(ctx->stream));
    double acc[AUG_N_STAGES] = {0};
    for (int c = 0; c < ctx->ev_n; ++c) {
        cudaEvent_t *ev = ctx->ev + (size_t)c * (2 * AUG_N_STAGES);
        for (int i = 0; i < AUG_N_STAGES; ++i) {
            float ms = 0.f;
            AUG_CUDA_OK(cudaEventElapsedTime(&ms, ev[2 * i], ev[2 * i + 1]));
            acc[i] += ms;
        }
    }
    for (int i = 0; i < AUG_N_STAGES; ++i) ms_host[i] = ctx->ev_n ? (float)(acc[i] / ctx->ev_n) : 0.f;
    if (n_calls_host) *n_calls_host = ctx->ev_n;
    ctx->ev_n = 0;
    return AUG_OK;
}

int64_t aug_launch_count(const AugCtx *ctx) { return ctx ? ctx->launches : 0; }

int aug_last_host_bytes(const AugCtx *ctx, int64_t *h2d_host, int64_t *d2h_host) {
    if (!ctx) return AUG_EINVAL;
    if (h2d_host) *h2d_host = ctx->last_h2d;
    if (d2h_host) *d2h_host = ctx->last_d2h;
    return AUG_OK;
}

}  // extern "C"
