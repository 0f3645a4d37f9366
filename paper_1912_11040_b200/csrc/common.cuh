// Internal declarations shared by the translation units of libaugb200.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/aug_b200.h"

namespace aug {

constexpr int CONV_BLK = 4096;          // output samples per convolution block
constexpr int CONV_F = 2 * CONV_BLK;    // real FFT size of one block
constexpr int CONV_N2 = CONV_F / 2;     // complex FFT size
constexpr int PARK_SMS = 160;       // multiprocessors that get parking slots in the fused convolution
constexpr int PARK_PER_SM = 3;      // slots per multiprocessor = resident CTAs of that kernel
constexpr int MAX_TAPS = 24576;
constexpr int MAX_ORDER = 32;
constexpr int MAX_HALF_W = 47;
constexpr int MAX_MEL = 128;

constexpr int EV_RING = 256;
#ifndef AUG_HOST_CHUNKS
#define AUG_HOST_CHUNKS 8
#endif
constexpr int HOST_CHUNKS = AUG_HOST_CHUNKS;   // pipeline depth of aug_pipeline_host

// How step 2 is run, fixed by the response length at aug_create:
//   ROUTE_FUSED_8192  rir_taps <= 8192: one partition of a 16384-point transform
//                     (16384 - taps + 1 outputs per block), one kernel
//   ROUTE_STORED      longer: partitions of 4096 taps, block spectra stored once and reused
enum Route { ROUTE_FUSED_8192 = 1, ROUTE_STORED = 2 };

enum Reason { R_NONE = 0, R_NSRC = 1, R_ORDER = 2, R_NOISE = 3 };

// Per-bin entry of the warped filterbank: the bin lies in edge interval `seg`
// (between edges e_seg and e_seg+1), at fraction `up` from its lower edge.
struct MelBin {
    float up;    // weight in filter seg   (rising side)
    float down;  // weight in filter seg-1 (falling side) = 1 - up
};

}  // namespace aug

struct AugCtx {
    AugConfig cfg;
    cudaStream_t stream;
    int device;
    int sm_count;          // multiprocessors of the device
    int smem_per_sm;       // shared memory of one multiprocessor, bytes
    int n_part;            // RIR partitions of CONV_BLK taps
    int route;             // aug::Route
    int n_bins;            // n_fft/2 + 1
    int t_cap;             // frames of an utterance of max_samples
    int64_t ws_stride;     // row stride (floats) of the y_s / v workspaces
    // device workspace (one allocation, carved up)
    void *ws_base;
    int64_t ws_bytes;
    float2 *tw;            // [TW_N] twiddles
    float *rir;            // [max_batch][max_sources][rir_taps]
    float2 *hspec;         // [max_batch][max_sources][n_part][CONV_N2]
    float2 *xspec;         // [max_batch][max_sources][nblk_cap][CONV_N2]; NULL unless route == ROUTE_STORED
    int nblk_cap;          // blocks of an utterance of max_samples
    float2 *park;          // [PARK_SMS * PARK_PER_SM][8192] products of noise sources waiting for the last one; NULL if unused
    int *park_flags;       // [PARK_SMS * PARK_PER_SM] 1 = slot taken
    int n_sm;              // multiprocessors with slots (PARK_SMS); CTAs on others sum in the time domain
    float *warped;         // [max_batch][ws_stride] speech after the waveform warp; NULL unless cfg.vtlp_win
    void *vtlp_tab;        // [max_batch][513] lower source bin (int), then [max_batch][513] fraction (float)
    float *ys;             // [max_batch][ws_stride]
    float *vv;             // [max_batch][ws_stride]
    double *energy;        // [max_batch][2]
    int *leff;             // [max_batch + 1] (last entry: largest over the batch)
    int *leff_seen;        // pinned host copy of that last entry from an earlier call (long-response contexts)
    int stored_only;       // this call launches the stored-spectra kernels alone taps up to the last non-zero one, largest over the utterance's sources
    float *gain;           // [max_batch] noise gain g for the requested SNR
    aug::MelBin *melw;     // [max_batch][n_bins]
    int *melstart;         // [max_batch][n_mel + 2]
    int *status;           // [2]: utterance, reason
    // instrumentation
    int64_t launches;      // kernels launched so far
    int timing;            // record events between the stages of aug_pipeline
    cudaEvent_t *ev;       // [EV_RING][2 * AUG_N_STAGES]: start and stop of every stage
    int ev_n;              // calls recorded
    // staging for the host-buffer entry point (NULL unless cfg.host_staging)
    float *st_speech;      // [max_batch][ws_stride]
    float *st_bank;        // [max_bank_samples]
    AugUttParams *st_table;
    int *st_lengths;
    float *st_feats;       // [max_batch][t_cap][n_mel]
    int *st_counts;
    int64_t last_h2d, last_d2h;                // bytes the last aug_pipeline_host call copied
    cudaStream_t s_side;                       // aug_pipeline builds the filterbank tables here, beside step 1
    cudaEvent_t ev_fork, ev_join;
    cudaStream_t s_h2d, s_d2h;                 // copy streams of the host-buffer entry point
    cudaStream_t s_h2d2;                       // the row-gather kernel's stream, beside the copy engine's
    cudaEvent_t ev_in[aug::HOST_CHUNKS], ev_out[aug::HOST_CHUNKS], ev_start;
    cudaEvent_t ev_in2[aug::HOST_CHUNKS], ev_len;
    int64_t bank_resident;                     // samples of st_bank filled by aug_upload_noise_bank (0 = none)
};

#define AUG_CUDA_OK(expr)                         \
    do {                                          \
        cudaError_t e__ = (expr);                 \
        if (e__ != cudaSuccess) return AUG_ECUDA; \
    } while (0)

// Let kernel Kern use as much dynamic shared memory as the device allows (the
// opt-in limit less the kernel's static shared memory).  The attribute belongs to
// the device's copy of the kernel, not to a context, so it is set once per device
// and to the largest value any configuration can ask for.
template <auto Kern>
inline int smem_opt_in(int device) {
    static std::atomic<unsigned long long> done{0};
    const unsigned long long bit = 1ull << (device & 63);
    if (done.load(std::memory_order_acquire) & bit) return AUG_OK;
    int optin = 0;
    cudaFuncAttributes fa;
    AUG_CUDA_OK(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device));
    AUG_CUDA_OK(cudaFuncGetAttributes(&fa, Kern));
    AUG_CUDA_OK(cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     optin - (int)fa.sharedSizeBytes));
    done.fetch_or(bit, std::memory_order_release);
    return AUG_OK;
}

// Launchers (defined next to their kernels).  They enqueue on ctx->stream unless a
// stream is passed.
int launch_rir(AugCtx *ctx, const AugUttParams *table, int B, float *rir, cudaStream_t st);
int launch_rir_spectra(AugCtx *ctx, const float *rir, const AugUttParams *table, int B,
                       cudaStream_t st);
// Convolution in two parts: `prepare` needs only the input audio (block spectra when
// the response has several partitions, else nothing), `finish` also needs the
// partition spectra of the impulse responses.
int launch_convolve_prepare(AugCtx *ctx, const float *speech, int64_t stride, const int *lengths,
                            const float *bank, int64_t bank_len, const AugUttParams *table, int B,
                            int max_len);
int launch_convolve_finish(AugCtx *ctx, const float *speech, int64_t stride, const int *lengths,
                           const float *bank, int64_t bank_len, const AugUttParams *table, int B,
                           int max_len);
int launch_mix(AugCtx *ctx, const int *lengths, const AugUttParams *table, int B, int max_len,
               float *wave_out, int64_t out_stride);
int launch_mel_tables(AugCtx *ctx, const AugUttParams *table, int B, cudaStream_t st);
int launch_vtlp_resynth(AugCtx *ctx, const float *speech, int64_t stride, const int *lengths,
                        const AugUttParams *table, int B, int max_len, float *out, int64_t out_stride);
int launch_stft_power(AugCtx *ctx, const float *wave, int64_t stride, const int *lengths, int B,
                      float *power, int T_max, int *counts);
int launch_logmel(AugCtx *ctx, const float *power, const int *counts, int B, int T_max,
                  float *feats);
int launch_fused_features(AugCtx *ctx, const int *lengths, const AugUttParams *table, int B,
                          float *feats, int T_max, int *counts, int max_len);
