/*
 * gen.c — seeded synthetic inputs (noise only; none of the attention / eviction arithmetic lives here).
 *
 * Every value is a pure function of (seed, tensor id, layer, sequence, head, index, channel), so any slice of any
 * tensor can be produced on its own and in any order. The counter is folded through the splitmix64 output function
 * and two such hashes feed a Box-Muller transform; a channel pair shares one transform (cosine for the even
 * channel, sine for the odd one).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

static inline uint64_t stream_key(uint64_t seed, uint32_t tensor, uint32_t layer, uint32_t seq, uint32_t head) {
    uint64_t h = mix64(seed);
    h = mix64(h ^ (uint64_t)tensor);
    h = mix64(h ^ (uint64_t)layer);
    h = mix64(h ^ (uint64_t)seq);
    h = mix64(h ^ (uint64_t)head);
    return h;
}

uint64_t wl_uniform_u64(uint64_t seed, uint32_t tensor, uint32_t layer, uint32_t seq, uint32_t head, uint64_t index) {
    return mix64(stream_key(seed, tensor, layer, seq, head) ^ mix64(index));
}

/* two standard normals for the channel pair (2*pair, 2*pair+1) of element `index` */
static inline void normal_pair(uint64_t skey, uint64_t index, uint32_t pair, double *a, double *b) {
    uint64_t h = mix64(skey ^ mix64((index << 12) | (uint64_t)pair));
    uint64_t h1 = mix64(h), h2 = mix64(h ^ 0xD1B54A32D192ED03ULL);
    double u1 = ((double)(h1 >> 11) + 1.0) * (1.0 / 9007199254740992.0); /* (0,1] */
    double u2 = (double)(h2 >> 11) * (1.0 / 9007199254740992.0);          /* [0,1) */
    double rad = sqrt(-2.0 * log(u1)), ang = 6.283185307179586476925 * u2;
    *a = rad * cos(ang);
    *b = rad * sin(ang);
}

/* out[n,d]: iid N(0,1); element index runs index0 .. index0+n-1 */
void wl_normal_block(uint64_t seed, uint32_t tensor, uint32_t layer, uint32_t seq, uint32_t head, uint64_t index0,
                     int64_t n, int32_t d, float *out) {
    uint64_t skey = stream_key(seed, tensor, layer, seq, head);
    for (int64_t i = 0; i < n; ++i)
        for (int32_t c = 0; c < d; c += 2) {
            double a, b;
            normal_pair(skey, index0 + (uint64_t)i, (uint32_t)(c >> 1), &a, &b);
            out[i * d + c] = (float)a;
            if (c + 1 < d) out[i * d + c + 1] = (float)b;
        }
}

/* out[n,d]: per-channel AR(1) chain x_0 = N_0, x_i = rho x_{i-1} + sigma N_i, chain index 0..n-1 */
void wl_ar1_chain(uint64_t seed, uint32_t tensor, uint32_t layer, uint32_t seq, uint32_t head, int64_t n, int32_t d,
                  double rho, double sigma, float *out) {
    uint64_t skey = stream_key(seed, tensor, layer, seq, head);
    double state[1024];
    if (d > 1024) return;
    for (int64_t i = 0; i < n; ++i)
        for (int32_t c = 0; c < d; c += 2) {
            double a, b;
            normal_pair(skey, (uint64_t)i, (uint32_t)(c >> 1), &a, &b);
            if (i == 0) { state[c] = a; if (c + 1 < d) state[c + 1] = b; }
            else { state[c] = rho * state[c] + sigma * a; if (c + 1 < d) state[c + 1] = rho * state[c + 1] + sigma * b; }
            out[i * d + c] = (float)state[c];
            if (c + 1 < d) out[i * d + c + 1] = (float)state[c + 1];
        }
}

/* in place: round float32 values to the nearest bf16 (ties to even), keeping them as float32 carriers */
void wl_round_bf16(float *a, int64_t n) {
    for (int64_t i = 0; i < n; ++i) {
        uint32_t x;
        memcpy(&x, a + i, 4);
        if ((x & 0x7f800000u) != 0x7f800000u) x += 0x7fffu + ((x >> 16) & 1u);
        x &= 0xffff0000u;
        memcpy(a + i, &x, 4);
    }
}
