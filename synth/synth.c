/*
 * Seeded synthetic inputs for structured-tensor workloads.
 *
 * Every value is a pure function of (seed, tensor id, logical dense linear index), so a slice of
 * a tensor can be produced without the rest of it, on any number of threads, with identical bits.
 * This file holds no index-map arithmetic: structured streams are produced by walking the index
 * domain with plain nested loops and a running counter.
 *
 * Hash: the SplitMix64 output function (Steele, Lea, Flood 2014; Vigna's public-domain constants).
 *   key = mix(seed * 256 + tensor_id),  h = mix(key ^ index)
 * Uniform:  m = h >> 40 (24 bits), value = (2m - 2^24) / 2^24, exactly representable in fp32,
 *           range [-1, 1).
 * Normal:   Box-Muller in double on u1 = (m + 0.5) / 2^24 and u2 = (mix(h) >> 40) / 2^24,
 *           multiplied by `scale` in double, rounded once to fp32.
 * bf16:     the fp32 value rounded to nearest-even on its upper 16 bits.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>

#define SYNTH_UNIFORM 0
#define SYNTH_NORMAL 1

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static inline uint64_t tensor_key(uint64_t seed, uint64_t tensor_id) {
    return mix64(seed * 256ull + tensor_id);
}

static inline float value_at(uint64_t key, int dist, double scale, uint64_t index) {
    uint64_t h = mix64(key ^ index);
    uint64_t m = h >> 40;
    if (dist == SYNTH_UNIFORM) {
        double v = ((double)(2 * (int64_t)m - (1 << 24))) / 16777216.0;
        return (float)(v * scale);
    }
    double u1 = ((double)m + 0.5) / 16777216.0;
    double u2 = (double)(mix64(h) >> 40) / 16777216.0;
    double z = sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * u2);
    return (float)(z * scale);
}

static inline uint16_t f32_to_bf16_rne(float f) {
    union { float f; uint32_t u; } c;
    c.f = f;
    uint32_t u = c.u;
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40u); /* NaN stays NaN */
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static inline void store_value(void* out, int as_bf16, size_t pos, float v) {
    if (as_bf16) ((uint16_t*)out)[pos] = f32_to_bf16_rne(v);
    else ((float*)out)[pos] = v;
}

/* Values of dense linear indices [first, first + n). */
void synth_fill_linear(uint64_t seed, uint64_t tensor_id, int dist, double scale, int as_bf16,
                       uint64_t first, uint64_t n, void* out) {
    uint64_t key = tensor_key(seed, tensor_id);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < (int64_t)n; ++t)
        store_value(out, as_bf16, (size_t)t, value_at(key, dist, scale, first + (uint64_t)t));
}

/* Row i of the full symmetric N x N matrix whose element (i, j) is keyed by the dense linear
 * index of (min(i,j), max(i,j)). */
void synth_fill_symmetric_row(uint64_t seed, uint64_t tensor_id, int dist, double scale,
                              int as_bf16, uint64_t N, uint64_t i, void* out) {
    uint64_t key = tensor_key(seed, tensor_id);
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < (int64_t)N; ++j) {
        uint64_t lo = i < (uint64_t)j ? i : (uint64_t)j;
        uint64_t hi = i < (uint64_t)j ? (uint64_t)j : i;
        store_value(out, as_bf16, (size_t)j, value_at(key, dist, scale, lo * N + hi));
    }
}

/* Upper triangle 0 <= i <= j < N of an N x N matrix (row stride N in the dense index space),
 * emitted row after row, j ascending.  Returns the number of values written; with out == NULL
 * nothing is written and the number of values is returned (counted by the same walk). */
uint64_t synth_stream_upper_triangle(uint64_t seed, uint64_t tensor_id, int dist, double scale,
                                     int as_bf16, uint64_t N, void* out) {
    uint64_t key = tensor_key(seed, tensor_id);
    uint64_t* start = (uint64_t*)malloc((N + 1) * sizeof(uint64_t));
    if (!start) return 0;
    start[0] = 0; /* running counter: where each row's values begin */
    for (uint64_t i = 0; i < N; ++i) start[i + 1] = start[i] + (N - i);
    if (!out) { uint64_t c = start[N]; free(start); return c; } /* size query */
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t i = 0; i < (int64_t)N; ++i)
        for (uint64_t j = (uint64_t)i; j < N; ++j)
            store_value(out, as_bf16, (size_t)(start[i] + (j - (uint64_t)i)),
                        value_at(key, dist, scale, (uint64_t)i * N + j));
    uint64_t total = start[N];
    free(start);
    return total;
}

/* Upper half cube 0 <= i < M, i <= j < N, 0 <= l < Q of an M x N x Q tensor, emitted in (i, j, l)
 * order.  Returns the number of values written (counted by the same walk when out == NULL). */
uint64_t synth_stream_upper_half_cube(uint64_t seed, uint64_t tensor_id, int dist, double scale,
                                      uint64_t M, uint64_t N, uint64_t Q, void* out) {
    uint64_t key = tensor_key(seed, tensor_id);
    uint64_t* start = (uint64_t*)malloc((M + 1) * sizeof(uint64_t));
    if (!start) return 0;
    start[0] = 0;
    for (uint64_t i = 0; i < M; ++i) start[i + 1] = start[i] + (i < N ? (N - i) * Q : 0);
    if (!out) { uint64_t c = start[M]; free(start); return c; }
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t i = 0; i < (int64_t)M; ++i)
        for (uint64_t j = (uint64_t)i; j < N; ++j)
            for (uint64_t l = 0; l < Q; ++l)
                store_value(out, 0, (size_t)(start[i] + (j - (uint64_t)i) * Q + l),
                            value_at(key, dist, scale, ((uint64_t)i * N + j) * Q + l));
    uint64_t total = start[M];
    free(start);
    return total;
}

/* Band |i - j| <= w of an N x N matrix emitted row after row, j ascending, nothing in between. */
uint64_t synth_stream_band_rows(uint64_t seed, uint64_t tensor_id, int dist, double scale, uint64_t N,
                                uint64_t w, void* out) {
    uint64_t key = tensor_key(seed, tensor_id);
    uint64_t* start = (uint64_t*)malloc((N + 1) * sizeof(uint64_t));
    if (!start) return 0;
    start[0] = 0;
    for (uint64_t i = 0; i < N; ++i) {
        uint64_t lo = i > w ? i - w : 0, hi = i + w < N - 1 ? i + w : N - 1;
        start[i + 1] = start[i] + (hi - lo + 1);
    }
    if (!out) { uint64_t c = start[N]; free(start); return c; }
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)N; ++i) {
        uint64_t ui = (uint64_t)i, lo = ui > w ? ui - w : 0, hi = ui + w < N - 1 ? ui + w : N - 1;
        for (uint64_t j = lo; j <= hi; ++j)
            store_value(out, 0, (size_t)(start[i] + (j - lo)), value_at(key, dist, scale, ui * N + j));
    }
    uint64_t total = start[N];
    free(start);
    return total;
}

/* Tetrahedron 0 <= i <= j <= k < n of an n x n x n tensor, emitted in (i, j, k) order. */
uint64_t synth_stream_tetrahedron(uint64_t seed, uint64_t tensor_id, int dist, double scale,
                                  int as_bf16, uint64_t n, void* out) {
    uint64_t key = tensor_key(seed, tensor_id);
    uint64_t* start = (uint64_t*)malloc((n + 1) * sizeof(uint64_t));
    if (!start) return 0;
    start[0] = 0; /* running counter: where each slab i begins */
    for (uint64_t i = 0; i < n; ++i) {
        uint64_t slab = 0;
        for (uint64_t j = i; j < n; ++j) slab += n - j;
        start[i + 1] = start[i] + slab;
    }
    if (!out) { uint64_t c = start[n]; free(start); return c; } /* size query */
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < (int64_t)n; ++i) {
        uint64_t pos = start[i];
        for (uint64_t j = (uint64_t)i; j < n; ++j)
            for (uint64_t k = j; k < n; ++k)
                store_value(out, as_bf16, (size_t)pos++,
                            value_at(key, dist, scale, ((uint64_t)i * n + j) * n + k));
    }
    uint64_t total = start[n];
    free(start);
    return total;
}

/* Band |i - j| <= w of an N x N matrix as 2w+1 diagonals of N slots each: diagonal d = j - i + w
 * (outer), row i (inner).  A slot whose column i + d - w falls outside [0, N) holds `pad_bits`
 * (a raw fp32 bit pattern, so a test can poison the padding).  Returns (2w+1) * N. */
uint64_t synth_stream_band_diagonals(uint64_t seed, uint64_t tensor_id, int dist, double scale,
                                     uint64_t N, uint64_t w, uint32_t pad_bits, float* out) {
    uint64_t key = tensor_key(seed, tensor_id);
    union { float f; uint32_t u; } pad;
    pad.u = pad_bits;
    for (uint64_t d = 0; d <= 2 * w; ++d) {
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < (int64_t)N; ++i) {
            int64_t j = i + (int64_t)d - (int64_t)w;
            out[d * N + (uint64_t)i] =
                (j < 0 || j >= (int64_t)N) ? pad.f
                                           : value_at(key, dist, scale, (uint64_t)i * N + (uint64_t)j);
        }
    }
    return (2 * w + 1) * N;
}
