// Host-side sampler of the per-utterance parameter table: the random room,
// reverberation time, positions, SNR and warp factor that the paper's simulator
// and VTLP draw per utterance (Sections 1 and 2.3).  Pure host code.
//
// Random numbers come from a counter-based generator: draw i of utterance b under
// `seed` is the SplitMix64 output function applied to seed + (b * 256 + i + 1) * gamma,
// so any row can be regenerated on its own and nothing depends on call order.
#include <math.h>
#include <string.h>

#include "common.cuh"

namespace {

inline uint64_t splitmix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

struct Draws {
    uint64_t seed;
    uint64_t row;
    uint32_t i;
    double uniform() {   // [0, 1)
        const uint64_t ctr = row * 256ull + (uint64_t)(i++) + 1ull;
        return (double)(splitmix64(seed + ctr * 0x9E3779B97F4A7C15ull) >> 11) * (1.0 / 9007199254740992.0);
    }
    double range(double lo, double hi) { return lo + (hi - lo) * uniform(); }
    int64_t integer(int64_t lo, int64_t hi) {   // inclusive
        if (hi <= lo) return lo;
        int64_t v = lo + (int64_t)floor(uniform() * (double)(hi - lo + 1));
        return v > hi ? hi : v;
    }
};

bool dist_ok(const AugDist *d) {
    for (int a = 0; a < 3; ++a)
        if (!(d->room_lo[a] > 0.f) || !(d->room_hi[a] >= d->room_lo[a])) return false;
    if (!(d->t60_lo > 0.f) || !(d->t60_hi >= d->t60_lo)) return false;
    if (d->order < 0 || d->order > aug::MAX_ORDER) return false;
    if (d->n_noise_lo < 0 || d->n_noise_hi < d->n_noise_lo || d->n_noise_hi > AUG_S_MAX - 1) return false;
    if (!(d->snr_hi >= d->snr_lo) || !(d->alpha_lo > 0.f) || !(d->alpha_hi >= d->alpha_lo) ||
        !(d->alpha_hi < 2.f))
        return false;
    if (!(d->wall_margin >= 0.f) || !(d->min_src_mic_dist >= 0.f)) return false;
    if (d->n_noise_hi > 0 && (d->bank_len < 1 || d->min_noise_len < 1)) return false;
    return true;
}

}  // namespace

extern "C" int aug_sample_params(uint64_t seed, const AugDist *dist, int B, const int *lengths_host,
                                 AugUttParams *table_host) {
    if (!dist || B < 0 || (B > 0 && (!lengths_host || !table_host))) return AUG_EINVAL;
    if (!dist_ok(dist)) return AUG_EINVAL;
    for (int b = 0; b < B; ++b) {
        if (lengths_host[b] < 0) return AUG_EINVAL;
        Draws rng{seed, (uint64_t)b, 0};
        AugUttParams r;
        memset(&r, 0, sizeof(r));
        double room[3];
        for (int a = 0; a < 3; ++a) {
            room[a] = rng.range(dist->room_lo[a], dist->room_hi[a]);
            r.room[a] = (float)room[a];
        }
        // Eyring: T60 = 0.161 V / (-S ln(1 - a)), beta = sqrt(1 - a), same on all six walls
        const double t60 = rng.range(dist->t60_lo, dist->t60_hi);
        const double vol = room[0] * room[1] * room[2];
        const double surf = 2.0 * (room[0] * room[1] + room[1] * room[2] + room[0] * room[2]);
        const float beta = (float)sqrt(exp(-0.161 * vol / (surf * t60)));
        for (int wl = 0; wl < 6; ++wl) r.beta[wl] = beta;
        double mic[3];
        for (int a = 0; a < 3; ++a) {
            const double m = fmin((double)dist->wall_margin, 0.25 * r.room[a]);
            mic[a] = rng.range(m, r.room[a] - m);
            r.mic[a] = (float)mic[a];
        }
        const int k = (int)rng.integer(dist->n_noise_lo, dist->n_noise_hi);
        r.n_src = 1 + k;
        r.order = dist->order;
        r.snr_db = (float)rng.range(dist->snr_lo, dist->snr_hi);
        r.alpha = (float)rng.range(dist->alpha_lo, dist->alpha_hi);
        for (int s = 0; s < r.n_src; ++s) {
            // redraw a source that lands too close to the microphone; the last try is
            // pushed away from it along x so the row is always valid
            for (int tries = 0; tries < 64; ++tries) {
                double d2 = 0.0;
                for (int a = 0; a < 3; ++a) {
                    const double m = fmin((double)dist->wall_margin, 0.25 * r.room[a]);
                    r.src_pos[s][a] = (float)rng.range(m, r.room[a] - m);
                    d2 += ((double)r.src_pos[s][a] - r.mic[a]) * ((double)r.src_pos[s][a] - r.mic[a]);
                }
                if (sqrt(d2) >= dist->min_src_mic_dist && d2 > 1e-6) break;
                if (tries == 63)
                    r.src_pos[s][0] = r.mic[0] < 0.5f * r.room[0] ? 0.75f * r.room[0] : 0.25f * r.room[0];
            }
        }
        const int64_t n = lengths_host[b];
        for (int j = 0; j < k; ++j) {
            int64_t hi = n < dist->bank_len ? n : dist->bank_len;
            if (hi < dist->min_noise_len) hi = dist->min_noise_len;
            if (hi > dist->bank_len) hi = dist->bank_len;
            int64_t lo = hi / 2 > dist->min_noise_len ? hi / 2 : dist->min_noise_len;
            if (lo > hi) lo = hi;
            int64_t len = rng.integer(lo, hi);
            int64_t off = rng.integer(0, dist->bank_len - len);
            if (len >= 4) {   // whole groups of four samples from a 16-byte boundary: 128-bit loads
                len &= ~(int64_t)3;
                off &= ~(int64_t)3;
            }
            r.noise_len[j] = (int32_t)len;
            r.noise_offset[j] = off;
            r.noise_weight[j] = 1.f;
        }
        table_host[b] = r;
    }
    return AUG_OK;
}
