/* Seeded synthetic inputs for the ICL-attention workloads.
 *
 * This module only draws numbers: it holds none of the method's arithmetic
 * (no scales, no FP8, no attention).  Both the CUDA library's tests and the
 * CPU oracle's tests are fed from the arrays it fills.
 *
 * Every element is a pure function of (seed, tensor id, b, h, row, column), so
 * any slice can be regenerated without materialising the rest:
 *   z      ~ N(0,1)   Box-Muller on a 64-bit hash of the element-pair counter
 *   gain_r = exp(sigma * n_r), n_r ~ N(0,1) per (tensor, b, h, row)   [optional]
 *   value  = z * gain_r * (outlier_gain if column is an outlier channel of (b,h))
 *            + shift
 *   stored as bf16, round-to-nearest-even.
 * The outlier channels of a head are the n_outlier columns with the smallest
 * hash of (seed, b, h, column); they are the same for every tensor of the head.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline uint64_t stream_key(uint64_t seed, uint64_t stream, uint64_t bh) {
    return mix64(mix64(mix64(seed) ^ (stream * 0xD6E8FEB86659FD93ull)) ^ bh);
}

/* two independent standard normals from one 64-bit hash */
static inline void normal_pair(uint64_t h, double* z0, double* z1) {
    double u1 = ((double)(h >> 32) + 0.5) * (1.0 / 4294967296.0);
    double u2 = ((double)(h & 0xFFFFFFFFull) + 0.5) * (1.0 / 4294967296.0);
    double r = sqrt(-2.0 * log(u1));
    double a = 6.283185307179586476925 * u2;
    *z0 = r * cos(a);
    *z1 = r * sin(a);
}

static inline uint16_t float_to_bf16_rne(float x) {
    uint32_t u;
    memcpy(&u, &x, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

typedef struct {
    uint16_t* out;
    uint64_t seed;
    int tensor_id;
    int B, H;
    int64_t R;
    int d;
    int n_outlier;
    double outlier_gain;
    double row_sigma;
    double shift;
    int64_t row_begin, row_end; /* rows of the flattened [B*H*R] axis */
} job_t;

static void outlier_mask(uint64_t seed, int64_t bh, int d, int n_outlier, uint8_t* mask) {
    memset(mask, 0, (size_t)d);
    uint64_t key = stream_key(seed, 1000, (uint64_t)bh);
    for (int pick = 0; pick < n_outlier && pick < d; ++pick) {
        int best = -1;
        uint64_t best_h = 0;
        for (int c = 0; c < d; ++c) {
            if (mask[c]) continue;
            uint64_t h = mix64(key ^ (uint64_t)c);
            if (best < 0 || h < best_h) { best = c; best_h = h; }
        }
        mask[best] = 1;
    }
}

static void* run_job(void* arg) {
    job_t* j = (job_t*)arg;
    int d = j->d;
    uint8_t* mask = (uint8_t*)malloc((size_t)d);
    int64_t cur_bh = -1;
    uint64_t key = 0, row_key = 0;
    for (int64_t fr = j->row_begin; fr < j->row_end; ++fr) {
        int64_t bh = fr / j->R;
        int64_t row = fr % j->R;
        if (bh != cur_bh) {
            cur_bh = bh;
            outlier_mask(j->seed, bh, d, j->n_outlier, mask);
            key = stream_key(j->seed, (uint64_t)j->tensor_id, (uint64_t)bh);
            row_key = stream_key(j->seed, 100 + (uint64_t)j->tensor_id, (uint64_t)bh);
        }
        double gain = 1.0;
        if (j->row_sigma != 0.0) {
            double n0, n1;
            normal_pair(mix64(row_key ^ (uint64_t)row), &n0, &n1);
            gain = exp(j->row_sigma * n0);
        }
        uint16_t* o = j->out + fr * d;
        for (int c = 0; c < d; c += 2) {
            uint64_t pair = ((uint64_t)row * (uint64_t)d + (uint64_t)c) >> 1;
            double z0, z1;
            normal_pair(mix64(key ^ (pair * 0x9E3779B97F4A7C15ull)), &z0, &z1);
            double v0 = z0 * gain * (mask[c] ? j->outlier_gain : 1.0) + j->shift;
            o[c] = float_to_bf16_rne((float)v0);
            if (c + 1 < d) {
                double v1 = z1 * gain * (mask[c + 1] ? j->outlier_gain : 1.0) + j->shift;
                o[c + 1] = float_to_bf16_rne((float)v1);
            }
        }
    }
    free(mask);
    return NULL;
}

/* Fill out[B,H,R,d] (bf16 bit patterns).  tensor_id: 0 Q_train, 1 K, 2 V,
 * 3 Q_test.  Returns 0. */
int workload_fill(uint16_t* out, uint64_t seed, int tensor_id, int B, int H,
                  int64_t R, int d, int n_outlier, double outlier_gain,
                  double row_sigma, double shift, int nthreads) {
    int64_t total = (int64_t)B * H * R;
    if (nthreads < 1) nthreads = 1;
    if (nthreads > 256) nthreads = 256;
    if ((int64_t)nthreads > total) nthreads = (int)(total > 0 ? total : 1);
    pthread_t th[256];
    job_t jobs[256];
    for (int t = 0; t < nthreads; ++t) {
        job_t* j = &jobs[t];
        j->out = out; j->seed = seed; j->tensor_id = tensor_id;
        j->B = B; j->H = H; j->R = R; j->d = d;
        j->n_outlier = n_outlier; j->outlier_gain = outlier_gain;
        j->row_sigma = row_sigma; j->shift = shift;
        j->row_begin = total * t / nthreads;
        j->row_end = total * (t + 1) / nthreads;
        pthread_create(&th[t], NULL, run_job, j);
    }
    for (int t = 0; t < nthreads; ++t) pthread_join(th[t], NULL);
    return 0;
}

/* The outlier-channel mask of head bh (for tests). */
void workload_outlier_mask(uint64_t seed, int64_t bh, int d, int n_outlier, uint8_t* mask) {
    outlier_mask(seed, bh, d, n_outlier, mask);
}
