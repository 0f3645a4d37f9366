/*
 * aug_b200 -- on-GPU speech augmentation and feature extraction (sm_100a).
 *
 * What the paper's CPU "example servers" do to every utterance before it
 * reaches a trainer (Sections 1 and 2.3: acoustic simulator with room
 * configurations and impulse responses made on the fly, noise at a random SNR,
 * VTLP with the bilinear warp of Eq. 1, mel filterbank features), done on one
 * GPU:
 *
 *   1. aug_rir_image_method  room impulse responses of a shoebox room
 *   2. aug_reverb_mix        reverberate speech and noise sources, mix at an SNR
 *   3. feat_stft_power       framing, Hann window, power spectrum
 *   4. feat_vtlp_logmel      warped mel filterbank, log (or power-law) compression
 *   *  aug_pipeline          1-4 in one call, intermediates kept on the device
 *
 * Conventions shared by all calls
 *   - Plain C ABI.  Every pointer is tagged `_dev` (device memory, caller-owned,
 *     16-byte aligned) or `_host`.  The library never frees or keeps a caller
 *     pointer beyond the kernels it enqueues.
 *   - All device work of a context is enqueued on the CUDA stream given to
 *     aug_create and the compute calls return without synchronising.  They
 *     allocate nothing: the context owns a workspace sized at aug_create.
 *   - Return value: AUG_OK (0) or a negative AugStatus.  Nothing throws, aborts
 *     or traps.  Rows of the parameter table that a kernel has to reject are
 *     recorded in a device status word, see aug_last_status.
 *   - Audio is fp32 at AugConfig.fs; sample counts and frame counts are int32;
 *     offsets into the noise bank are int64.
 *   - A context serialises its work on its one stream and reuses one workspace:
 *     use it from one host thread at a time; several contexts (one per thread or
 *     per stream) are independent.  Use a context on the device it was created on.
 */
#ifndef AUG_B200_H
#define AUG_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AUG_S_MAX 4 /* speech + at most three noise sources per utterance */

typedef enum {
    AUG_OK = 0,
    AUG_EINVAL = -1, /* null or misaligned pointer, bad scalar argument */
    AUG_ECAP = -2,   /* batch, length, frames, taps or order beyond the context's capacity */
    AUG_ECUDA = -3,  /* a CUDA runtime call or kernel launch failed */
    AUG_EPARAM = -4, /* a parameter-table row failed validation */
    AUG_ENOMEM = -5  /* workspace allocation failed in aug_create */
} AugStatus;

typedef enum { AUG_COMPRESS_LOG = 0, AUG_COMPRESS_POW_1_15 = 1 } AugCompression;

/* Which image sources a reflection order N keeps: those reached by at most N
 * reflections in total (|kx|+|ky|+|kz| <= N, the default), or the whole cube
 * max(|kx|,|ky|,|kz|) <= N, up to 3N reflections: (2N+1)^3 images, a stress mode. */
typedef enum { AUG_LATTICE_TOTAL = 0, AUG_LATTICE_CUBE = 1 } AugLattice;

/* Rows of the host feature buffer that aug_pipeline_host writes.  PADDED (default): all
 * T_max rows of every utterance, those at and beyond its frame count holding pad_value.
 * VALID: only the frame_counts[b] rows that hold features; the other rows of the caller's
 * buffer are left as they are (a caller that packs by frame count, or keeps a buffer it
 * filled with its pad value once, saves the transfer of the padding: Section 2.4's
 * concern is keeping the trainer fed). */
typedef enum { AUG_HOST_ROWS_PADDED = 0, AUG_HOST_ROWS_VALID = 1 } AugHostRows;

/* Fixed at aug_create.  Plain data, no pointers. */
typedef struct {
    int32_t fs;              /* sampling rate, Hz */
    int32_t win;             /* window length in samples (<= n_fft) */
    int32_t hop;             /* frame shift in samples */
    int32_t n_fft;           /* DFT size K: 512 or 1024 */
    int32_t n_mel;           /* mel bands M, 1..128 */
    float f_lo;              /* lowest filterbank edge, Hz */
    float f_hi;              /* highest filterbank edge, Hz */
    int32_t rir_taps;        /* L: taps of every impulse response, 1..24576 */
    int32_t max_order;       /* largest reflection order a row may ask for, 0..32 */
    int32_t max_sources;     /* 1..AUG_S_MAX */
    int32_t frac_half_width; /* W_h of the windowed-sinc delay kernel, 1..47 */
    float sound_speed;       /* m/s */
    float log_floor;         /* filterbank energies are clamped to this before compression */
    float pad_value;         /* written to feature rows at and beyond the frame count */
    int32_t compression;     /* AugCompression */
    int32_t max_batch;       /* capacity: utterances per call */
    int32_t max_samples;     /* capacity: samples per utterance */
    int32_t host_staging;    /* non-zero: also allocate device staging for aug_pipeline_host */
    int32_t image_lattice;   /* AugLattice */
    int64_t max_bank_samples; /* capacity of the staged noise bank (host_staging only) */
    int32_t vtlp_win;        /* 0: the warp of Eq. 1 acts inside the mel filterbank (default).
                                > 0: it is applied to the speech waveform before the simulator,
                                with this window (samples; a multiple of 4, at most 1024; 800 is
                                the 50 ms of Section 4) and the filterbank stays unwarped */
    int32_t host_rows;       /* AugHostRows: what aug_pipeline_host writes to the host feature buffer */
} AugConfig;

/*
 * One row per utterance, 160 bytes.  Drawn on the HOST (the random room, SNR and
 * warp factor of Sections 1 / 2.3) and copied to the device by the caller.
 */
typedef struct {
    float room[3];                 /* shoebox side lengths, metres */
    float beta[6];                 /* wall reflection coefficients in [0,1]: x=0, x=Lx, y=0, y=Ly, z=0, z=Lz */
    float mic[3];                  /* microphone position */
    int32_t n_src;                 /* 1 + number of noise sources, 1..max_sources */
    int32_t order;                 /* keep images with |kx|+|ky|+|kz| <= order */
    float snr_db;                  /* power of reverberant speech over power of summed reverberant noise */
    float alpha;                   /* VTLP warp factor of Eq. 1, in (0,2); 1 = no warp */
    float src_pos[AUG_S_MAX][3];   /* [0] = speech source, [1..] = noise sources */
    int64_t noise_offset[AUG_S_MAX - 1]; /* start of this source's stretch of the noise bank */
    int32_t noise_len[AUG_S_MAX - 1];    /* its length; it repeats end to end over the utterance.
                                            Any offset and length work; stretches whose offset and
                                            length are multiples of 4 samples are read with 128-bit
                                            loads and convolve faster */
    float noise_weight[AUG_S_MAX - 1];   /* relative level of this source in the noise sum */
} AugUttParams;

typedef struct AugCtx AugCtx; /* opaque: configuration, tables, workspace */

/* -------------------------------------------------------------- host-only helpers */

/* Message for a status code; never NULL; static storage. */
const char *aug_strerror(int code);

/* Frames of an utterance of n_samples: 1 + (n_samples - win) / hop when
 * n_samples >= win, else 0 (no padding, no centring).  Pure integer arithmetic;
 * the kernels use the same expression. */
int aug_frame_count(int n_samples, int win, int hop);

/* Bytes of device workspace a context of this configuration allocates, or a
 * negative AugStatus if the configuration is invalid. */
int64_t aug_workspace_bytes(const AugConfig *cfg_host);

/* Check B host rows against cfg: finite values, room sides > 0, microphone and
 * sources inside the room and not coincident, beta in [0,1], alpha in (0,2),
 * n_src in [1,max_sources], order in [0,max_order], noise stretches inside
 * [0,bank_len) with positive length.  Returns AUG_OK or AUG_EPARAM with the index
 * of the first bad row in *bad_row_host (may be NULL). */
int aug_validate_params(const AugConfig *cfg_host, const AugUttParams *table_host, int B,
                        int64_t bank_len, int *bad_row_host);

/* Ranges the per-utterance parameters are drawn from (uniformly, independently):
 * the variety of room sizes, reverberation times and SNRs that Section 1 describes
 * for the simulator, and the random warp factor of Section 2.3. */
typedef struct {
    float room_lo[3], room_hi[3]; /* shoebox side lengths, metres */
    float t60_lo, t60_hi;         /* reverberation time, seconds; turned into one wall reflection
                                     coefficient by Eyring's formula */
    int32_t order;                /* reflection order written to every row */
    int32_t n_noise_lo, n_noise_hi; /* noise sources per utterance, 0..AUG_S_MAX-1 */
    float snr_lo, snr_hi;         /* dB */
    float alpha_lo, alpha_hi;     /* VTLP warp factor (Table 2 of the paper tries 0.8..1.2) */
    float wall_margin;            /* microphone and sources keep this distance from the walls */
    float min_src_mic_dist;       /* sources are redrawn while closer than this to the microphone */
    int32_t min_noise_len;        /* shortest stretch of the noise bank a source may loop */
    int64_t bank_len;             /* samples in the noise bank the offsets refer to */
} AugDist;

/* Draw B rows on the host from `seed` (counter-based SplitMix64: row b depends only
 * on seed and b).  Each noise source gets a stretch of the bank of length between
 * half the utterance and the whole utterance (clamped to [min_noise_len, bank_len])
 * at a uniform offset, weight 1; offset and length are rounded down to multiples of 4
 * samples (lengths of at least 4) so that the stretches can be read with 128-bit loads.
 * Rows always pass aug_validate_params for a
 * configuration with max_order >= order and max_sources > n_noise_hi.
 * Returns AUG_EINVAL for null pointers or inconsistent ranges. */
int aug_sample_params(uint64_t seed, const AugDist *dist_host, int B, const int *lengths_host,
                      AugUttParams *table_host);

/* -------------------------------------------------------------- context */

/* Create a context for cfg on the current CUDA device; cuda_stream is a
 * cudaStream_t (NULL = default stream).  All allocation happens here.
 * On failure *out is NULL. */
int aug_create(AugCtx **out, const AugConfig *cfg_host, void *cuda_stream);

/* Waits for the context's stream, frees the workspace.  NULL is accepted. */
int aug_destroy(AugCtx *ctx);

/* Synchronises the context's stream and reads the device status word.
 * *utt_host = first utterance a kernel rejected (-1 if none), *reason_host =
 * 1 n_src out of range, 2 order out of range, 3 bad noise stretch (the kernels
 * contain no waits on other blocks, so nothing else can go wrong on the device
 * short of a launch failure).  A rejected utterance gets zero impulse
 * responses / silent output; nothing faults.  The word is cleared by the read. */
int aug_last_status(AugCtx *ctx, int *utt_host, int *reason_host);

/* -------------------------------------------------------------- before step 1 (optional)
 * VTLP on the waveform with resynthesis (Section 2.3: the warp of Eq. 1 is applied to
 * the speech before the acoustic simulator, so that noise and reverberation are not
 * warped; Section 4 finds a 50 ms window best).  The paper prints only the frequency
 * map; what is computed here: frames of vtlp_win samples every vtlp_win/4, periodic
 * Hann, the utterance zero-padded by 3 vtlp_win/4 in front; 1024-point DFT; the
 * spectrum at bin k becomes the old spectrum at the frequency that Eq. 1 moves to
 * bin k, by linear interpolation between the two nearest bins; inverse DFT, first
 * vtlp_win samples, Hann again, overlap-add, division by the summed squared windows.
 * alpha = 1 returns the input.
 *   speech_dev [B][stride] -> warped_dev [B][out_stride], samples [0, lengths[b]) written
 * Needs a context created with vtlp_win > 0 (AUG_EINVAL otherwise).  aug_pipeline of
 * such a context runs this on the speech first and builds the filterbank unwarped. */
int aug_vtlp_resynth(AugCtx *ctx, const float *speech_dev, int64_t stride, const int *lengths_dev,
                     const AugUttParams *table_dev, int B, float *warped_dev, int64_t out_stride);

/* -------------------------------------------------------------- step 1
 * Room impulse responses by the image-source method (simulator block, Sections
 * 1 and 2.3; computed on the fly per utterance as Section 1 requires).
 *   rir_dev [B][max_sources][rir_taps] fp32, overwritten; sources >= n_src get zeros.
 * For each source the sum runs over the image lattice |kx|+|ky|+|kz| <= order
 * (or the cube, see AugLattice);
 * an image at distance d adds (prod beta^hits / d) times a Hann-windowed sinc
 * (half width frac_half_width) centred at d*fs/sound_speed samples.
 * Microphone arrays (the two microphones 6.8 cm apart of the far-field experiment
 * in Section 4): a row describes ONE microphone.  For C channels the caller passes
 * C rows per utterance -- row C*u + c is channel c of utterance u -- that differ
 * only in `mic`, with the speech row and length repeated, and reads channel c from
 * row C*u + c of every output.  Each row is mixed at the row's snr_db on its own. */
int aug_rir_image_method(AugCtx *ctx, const AugUttParams *table_dev, int B, float *rir_dev);

/* -------------------------------------------------------------- step 2
 * Reverberation and noise mixing (simulator block, Sections 1 and 2.3).
 *   speech_dev  [B][speech_stride] fp32; speech_stride a multiple of 4
 *   lengths_dev [B] int32, 0 <= lengths[b] <= min(speech_stride, max_samples)
 *   noise_bank_dev [bank_len] fp32 (may be NULL when no row has noise)
 *   rir_dev     as written by step 1
 *   wave_out_dev [B][speech_stride] fp32: samples [0,lengths[b]) written,
 *               the rest of each row left untouched
 * y_s = speech * rir[0] and v = sum_k weight_k (noise_k * rir[k]) are causal
 * convolutions cut to the utterance length, done as FFT overlap convolution (the
 * block size follows the last non-zero tap of an utterance's responses, so zero
 * tails of the response buffers cost nothing);
 * out = y_s + g v with g = sqrt(sum y_s^2 / (sum v^2 10^(snr_db/10))), g = 0 when
 * there is no noise or either sum is zero. */
int aug_reverb_mix(AugCtx *ctx, const float *speech_dev, int64_t speech_stride,
                   const int *lengths_dev, const float *noise_bank_dev, int64_t bank_len,
                   const float *rir_dev, const AugUttParams *table_dev, int B,
                   float *wave_out_dev);

/* -------------------------------------------------------------- step 3
 * Framing, periodic Hann window and power spectrum (feature block, Section 2.3).
 *   wave_dev  [B][stride] fp32;  power_dev [B][T_max][n_fft/2+1] fp32
 *   frame_counts_dev [B] int32 = min(aug_frame_count(lengths[b]), T_max)
 * P[t][k] = |sum_{n<win} hann[n] wave[t hop + n] exp(-2 pi i k n / n_fft)|^2, no
 * scaling.  Rows t >= frame count are set to zero. */
int feat_stft_power(AugCtx *ctx, const float *wave_dev, int64_t stride, const int *lengths_dev,
                    int B, float *power_dev, int T_max, int *frame_counts_dev);

/* -------------------------------------------------------------- step 4
 * Mel filterbank with the VTLP warp of Eq. 1 and compression (Section 2.3).
 *   feats_dev [B][T_max][n_mel] fp32
 * Triangles are linear in mel (2595 log10(1+f/700)), peak 1, edges equally spaced
 * from f_lo to f_hi, evaluated at the warped frequency of each DFT bin
 * (omega' of Eq. 1 with the row's alpha).  feat = ln(max(E, log_floor)), or
 * max(E, log_floor)^(1/15) for AUG_COMPRESS_POW_1_15.  Rows t >= frame_counts[b]
 * receive pad_value. */
int feat_vtlp_logmel(AugCtx *ctx, const float *power_dev, const int *frame_counts_dev,
                     const AugUttParams *table_dev, int B, int T_max, float *feats_dev);

/* -------------------------------------------------------------- step 4, allocation-free
 * (an addition of this library; the paper has no counterpart)
 *
 * The same computation as feat_vtlp_logmel for callers that cannot allocate
 * device memory and therefore cannot own an AugCtx (aug_create calls cudaMalloc):
 * code embedded in an application whose memory pool already holds the whole
 * device, latency-critical front-ends that must stay off the allocator once
 * running, or components that are only ever handed device pointers and a stream.
 * The per-utterance filterbank tables the kernels need are kept in a fixed array
 * built into the library (about 1.13 MiB; every GPU that loads the library holds
 * it until the process exits).  This call and everything it calls performs no
 * cudaMalloc / cudaFree and uses no allocating library.
 *
 *   cfg_host     only n_fft, n_mel, fs, f_lo, f_hi, log_floor, pad_value and
 *                compression are read
 *   power_dev, frame_counts_dev, table_dev, feats_dev, T_max: as feat_vtlp_logmel
 *   cuda_stream  cudaStream_t to enqueue on (NULL = default stream); returns
 *                without synchronising
 *
 * Limits: B <= AUG_NOALLOC_MAX_BATCH and n_mel <= 128, else AUG_ECAP ("request
 * exceeds the capacity ..."); n_fft must be 512 or 1024, else AUG_EINVAL.  Larger
 * batches must be split by the caller.
 * First call on a device: it looks up the device address of the built-in array
 * (cudaGetSymbolAddress, once per device, with that device current).  Make that
 * first call during start-up, before any stream capture is begun.
 * Sharing: all calls in the process use the one array on a device and it keeps
 * whatever the last call wrote.  Each call rewrites the part it reads, so stale
 * contents are never used, but two calls that can run at the same time on the
 * GPU (different streams, different host threads) race on it: serialise them. */
#define AUG_NOALLOC_MAX_BATCH 256
int feat_vtlp_logmel_noalloc(const AugConfig *cfg_host, const float *power_dev,
                             const int *frame_counts_dev, const AugUttParams *table_dev, int B,
                             int T_max, float *feats_dev, void *cuda_stream);

/* -------------------------------------------------------------- after the features
 * Cepstra: orthonormal DCT-II of each feature row (the MFCC baseline of Table 1
 * when the features are log-mel):  c_i = s_i sum_m x[m] cos(pi i (m + 1/2) / n_mel),
 * s_0 = sqrt(1/n_mel), s_i = sqrt(2/n_mel), i < n_cep <= n_mel.
 *   feats_dev [B][T_max][n_mel] -> mfcc_dev [B][T_max][n_cep]; rows t >= frame_counts[b]
 *   receive pad_value. */
int feat_mfcc(AugCtx *ctx, const float *feats_dev, const int *frame_counts_dev, int B, int T_max,
              int n_cep, float *mfcc_dev);

/* Per-utterance mean and (population) variance of each of D features over the
 * frame_counts[b] valid frames: mean_dev, var_dev [B][D]; both 0 for an utterance
 * without frames.  Sums are carried in fp64. */
int feat_mean_var(AugCtx *ctx, const float *feats_dev, const int *frame_counts_dev, int B, int T_max,
                  int D, float *mean_dev, float *var_dev);

/* Host only.  Padded batches of similar length (Section 2.2): perm_host[B] lists the
 * utterances by increasing length (stable), so consecutive groups of `batch` entries
 * pad least; batch_max_host[ceil(B/batch)] (may be NULL) receives each group's
 * longest length. */
int aug_bucket_by_length(const int *lengths_host, int B, int batch, int *perm_host,
                         int *batch_max_host);

/* -------------------------------------------------------------- steps 1-4
 * The whole path for a batch.  Arguments as above; additionally
 *   lengths_host  the same lengths in host memory (may be NULL): used only to size
 *                 launches tightly and to check capacities without a device sync
 *   wave_out_dev_or_null  if not NULL, also receives the mixed waveform as in step 2
 * Writes feats_dev [B][T_max][n_mel] (padded with pad_value) and frame_counts_dev. */
int aug_pipeline(AugCtx *ctx, const float *speech_dev, int64_t speech_stride,
                 const int *lengths_dev, const int *lengths_host, const float *noise_bank_dev,
                 int64_t bank_len, const AugUttParams *table_dev, int B, float *feats_dev,
                 int T_max, int *frame_counts_dev, float *wave_out_dev_or_null);

/* Same call for callers that hold HOST buffers (the context must have been created
 * with host_staging).  Inputs are copied to device staging owned by the context,
 * the path runs, feats ([B][T_max][n_mel]; all rows, padded, or with
 * AugConfig.host_rows = AUG_HOST_ROWS_VALID only the first frame_counts[b] rows of
 * every utterance, the rest of the buffer untouched) and frame counts are copied
 * back, and the call returns after synchronising, so the host buffers are free
 * again.  The longest rows of a chunk go by the copy engine while the kernel fetches
 * the others, and valid feature rows are written by a kernel straight into a pinned
 * (mapped) feature buffer, else by one copy per utterance.  Internally the batch is cut into up to 8 chunks of utterances that are
 * copied in, computed and copied out concurrently on three streams; speech rows
 * are copied only up to their length when that saves more than the extra copy
 * calls cost.  Host buffers should be pinned: copies then run asynchronously, and
 * the ragged rows of a pinned (mapped) speech buffer are fetched by one small kernel
 * per chunk that reads host memory directly instead of one copy per row.
 * noise_bank_host may be NULL with bank_len > 0
 * when a bank of exactly bank_len samples was uploaded with aug_upload_noise_bank:
 * that copy is then used and nothing of the bank crosses the bus (AUG_EINVAL if
 * there is none or its length differs). */
int aug_pipeline_host(AugCtx *ctx, const float *speech_host, int64_t speech_stride,
                      const int *lengths_host, const float *noise_bank_host, int64_t bank_len,
                      const AugUttParams *table_host, int B, float *feats_host, int T_max,
                      int *frame_counts_host);

/* A noise database that stays the same from batch to batch need not be sent with
 * every aug_pipeline_host call: copy bank_len samples into the context's device
 * staging once (host_staging contexts only, bank_len <= max_bank_samples; the call
 * synchronises, so the host buffer is free on return).  The copy stays valid until
 * the next aug_upload_noise_bank or the next aug_pipeline_host call that passes a
 * bank pointer of its own.  (Interface of this library; the paper's example servers
 * keep their noise database in host memory.) */
int aug_upload_noise_bank(AugCtx *ctx, const float *noise_bank_host, int64_t bank_len);

/* -------------------------------------------------------------- measurement utilities
 * (instrumentation of this library; the paper has no counterpart) */

#define AUG_N_STAGES 7 /* 0 impulse responses, 1 response lengths and spectra, 2 filterbank tables
                            (on a stream of their own beside stages 0 and 1: their time is the
                            time they took there and is not part of the sum of the others),
                          3 waveform warp (vtlp_win > 0) and block spectra of the audio (contexts
                            sized for responses of more than 8192 taps),
                          4 convolution, 5 waveform mix (only when requested), 6 features */

/* The fused convolution (responses of up to 8192 taps) sums several noise sources of an
 * utterance in the frequency domain through parking slots in the workspace, three per
 * multiprocessor; a CTA that finds none free sums in the time domain instead.
 * hold != 0 marks every slot taken, so that this second way can be exercised and
 * timed; hold == 0 frees them.  Synchronises the stream; call it only between
 * pipeline calls. */
int aug_hold_parking_slots(AugCtx *ctx, int hold);

/* on != 0: aug_pipeline records CUDA events between its kernels (up to 256 calls
 * are kept); on == 0: stop.  Either way the record is cleared. */
int aug_enable_stage_timing(AugCtx *ctx, int on);

/* Synchronises the stream; ms_host[AUG_N_STAGES] = mean device time of each stage
 * over the recorded aug_pipeline calls, *n_calls_host = how many; clears the record. */
int aug_stage_times(AugCtx *ctx, float *ms_host, int *n_calls_host);

/* Kernels this context has launched since aug_create. */
int64_t aug_launch_count(const AugCtx *ctx);

/* Bytes the last aug_pipeline_host call copied host-to-device and device-to-host. */
int aug_last_host_bytes(const AugCtx *ctx, int64_t *h2d_host, int64_t *d2h_host);

/* Runs a register-resident FMA loop on every SM of the current device and writes
 * the best of three fp32 rates (TFLOP/s, 2 flop per FMA) to *tflops_host.
 * Synchronises cuda_stream. */
int aug_measure_fp32_peak(void *cuda_stream, float *tflops_host);

#ifdef __cplusplus
}
#endif
#endif /* AUG_B200_H */
