/* Seeded synthetic inputs: graphs and tensors.
 *
 * This file holds no message-passing arithmetic.  It only produces inputs:
 * COO edge lists (source vector + target vector, the default topology format
 * of Sec. 3 "Graph Data Structures") and feature / weight tensors.  The same
 * host arrays are handed to the CPU checker and to the GPU library.
 *
 * Every random number is a pure function of (seed, stream, counter), so a
 * generator gives the same bytes on every machine and with any thread count.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC synth.c -o libgnn_synth.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z) {
    /* splitmix64 output function (Steele, Lea, Flood 2014) */
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

uint64_t synth_u64(uint64_t seed, uint64_t stream, uint64_t ctr) {
    uint64_t k = mix64(seed + 0x9E3779B97F4A7C15ULL * (stream + 1));
    return mix64(k + 0x9E3779B97F4A7C15ULL * (ctr + 1));
}

/* uniform in (0,1): 53 random bits, never 0 */
static inline double u01(uint64_t seed, uint64_t stream, uint64_t ctr) {
    return ((double)(synth_u64(seed, stream, ctr) >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

/* uniform integer in [0, range) by multiply-high */
static inline uint64_t ubelow(uint64_t r, uint64_t range) {
    return (uint64_t)(((__uint128_t)r * (__uint128_t)range) >> 64);
}

static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* standard normal: Box-Muller in fp64; element i uses counters 2i and 2i+1 */
static inline double normal_at(uint64_t seed, uint64_t stream, uint64_t i) {
    double u1 = u01(seed, stream, 2 * i), u2 = u01(seed, stream, 2 * i + 1);
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * u2);
}

void synth_fill_normal_f32(float* out, int64_t n, uint64_t seed, uint64_t stream) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = (float)normal_at(seed, stream, (uint64_t)i);
}

/* bf16 tensor = the fp32 tensor of the same (seed, stream), rounded to nearest even */
void synth_fill_normal_bf16(uint16_t* out, int64_t n, uint64_t seed, uint64_t stream) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        out[i] = f32_to_bf16_rne((float)normal_at(seed, stream, (uint64_t)i));
}

void synth_fill_uniform_f32(float* out, int64_t n, double lo, double hi, uint64_t seed,
                            uint64_t stream) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        out[i] = (float)(lo + (hi - lo) * u01(seed, stream, (uint64_t)i));
}

/* ---- G(n, M): M distinct unordered pairs u != v, both directions emitted ----
 * Edge 2t is (u,v), edge 2t+1 is (v,u), in the order the pairs were accepted.
 * Returns the number of directed edges written (2*pairs). */
int64_t synth_gnm(int32_t n, int64_t pairs, uint64_t seed, int32_t* src, int32_t* dst) {
    if (n < 2) return 0;
    int64_t maxpairs = (int64_t)n * (n - 1) / 2;
    if (pairs > maxpairs) pairs = maxpairs;
    /* open-addressing set of accepted pairs keyed by lo*n+hi */
    uint64_t cap = 16;
    while (cap < (uint64_t)pairs * 3 + 16) cap <<= 1;
    int64_t* tab = (int64_t*)malloc(cap * sizeof(int64_t));
    for (uint64_t i = 0; i < cap; ++i) tab[i] = -1;
    int64_t got = 0;
    uint64_t ctr = 0;
    while (got < pairs) {
        int32_t u = (int32_t)ubelow(synth_u64(seed, 1, ctr), (uint64_t)n);
        int32_t v = (int32_t)ubelow(synth_u64(seed, 2, ctr), (uint64_t)n);
        ++ctr;
        if (u == v) continue;
        int32_t lo = u < v ? u : v, hi = u < v ? v : u;
        int64_t key = (int64_t)lo * n + hi;
        uint64_t h = mix64((uint64_t)key) & (cap - 1);
        int dup = 0;
        while (tab[h] != -1) {
            if (tab[h] == key) { dup = 1; break; }
            h = (h + 1) & (cap - 1);
        }
        if (dup) continue;
        tab[h] = key;
        src[2 * got] = u;     dst[2 * got] = v;
        src[2 * got + 1] = v; dst[2 * got + 1] = u;
        ++got;
    }
    free(tab);
    return 2 * got;
}

/* ---- batch of G small graphs, block-diagonal (Sec. 3: batching of small graphs) ----
 * graph g has n_g ~ U{nmin..nmax} nodes; every unordered pair inside a graph is kept
 * with probability p and emitted in both directions.  graph_ptr[G+1] gets the node
 * offsets.  Returns directed edges written, or -1 if cap is too small. */
int64_t synth_batched_er(int32_t G, int32_t nmin, int32_t nmax, double p, uint64_t seed,
                         int32_t* graph_ptr, int32_t* src, int32_t* dst, int64_t cap) {
    int64_t e = 0;
    int32_t off = 0;
    graph_ptr[0] = 0;
    for (int32_t g = 0; g < G; ++g) {
        int32_t ng = nmin + (int32_t)ubelow(synth_u64(seed, 3, (uint64_t)g), (uint64_t)(nmax - nmin + 1));
        uint64_t c = 0;
        for (int32_t u = 0; u < ng; ++u)
            for (int32_t v = u + 1; v < ng; ++v) {
                double r = u01(seed, 1000 + (uint64_t)g, c++);
                if (r < p) {
                    if (e + 2 > cap) return -1;
                    src[e] = off + u; dst[e] = off + v; ++e;
                    src[e] = off + v; dst[e] = off + u; ++e;
                }
            }
        off += ng;
        graph_ptr[g + 1] = off;
    }
    return e;
}

/* ---- preferential attachment: m0 = m+1 clique seed, each new node attaches to m
 * distinct existing nodes chosen in proportion to degree (uniform draw from the
 * running endpoint list, duplicates redrawn).  Both directions are emitted.
 * Returns directed edges = 2*(m0*(m0-1)/2 + m*(n-m0)). */
int64_t synth_barabasi_albert(int32_t n, int32_t m, uint64_t seed, int32_t* src, int32_t* dst) {
    int32_t m0 = m + 1;
    if (n < m0) return 0;
    int64_t und = (int64_t)m0 * (m0 - 1) / 2 + (int64_t)m * (n - m0);
    int32_t* ends = (int32_t*)malloc((size_t)(2 * und) * sizeof(int32_t));
    int64_t ne = 0, e = 0;
    for (int32_t u = 0; u < m0; ++u)
        for (int32_t v = u + 1; v < m0; ++v) {
            src[e] = u; dst[e] = v; ++e;
            src[e] = v; dst[e] = u; ++e;
            ends[ne++] = u; ends[ne++] = v;
        }
    int32_t pick[64];
    uint64_t ctr = 0;
    for (int32_t v = m0; v < n; ++v) {
        int k = 0;
        while (k < m) {
            int32_t t = ends[ubelow(synth_u64(seed, 4, ctr++), (uint64_t)ne)];
            int dup = 0;
            for (int q = 0; q < k; ++q) dup |= (pick[q] == t);
            if (!dup) pick[k++] = t;
        }
        for (int q = 0; q < m; ++q) {
            src[e] = v; dst[e] = pick[q]; ++e;
            src[e] = pick[q]; dst[e] = v; ++e;
            ends[ne++] = v; ends[ne++] = pick[q];
        }
    }
    free(ends);
    return e;
}

/* ---- R-MAT (Chakrabarti, Zhan, Faloutsos 2004), quadrant probabilities a,b,c,(1-a-b-c),
 * no noise.  Pair t is redrawn (attempt counter) while an endpoint >= nlimit or u == v.
 * symmetric != 0: pair t gives edges 2t = (u,v) and 2t+1 = (v,u); else edge t = (u,v).
 * Duplicates are kept. */
void synth_rmat(int32_t scale, int32_t nlimit, int64_t pairs, double a, double b, double c,
                int32_t symmetric, uint64_t seed, int32_t* src, int32_t* dst) {
    const uint32_t ta = (uint32_t)(a * 65536.0), tb = (uint32_t)((a + b) * 65536.0),
                   tc = (uint32_t)((a + b + c) * 65536.0);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < pairs; ++t) {
        uint64_t ctr = 0;
        int32_t u, v;
        for (;;) {
            u = 0; v = 0;
            uint64_t word = 0;
            for (int32_t lvl = 0; lvl < scale; ++lvl) {
                if ((lvl & 3) == 0) word = synth_u64(seed, 0x100000000ULL + (uint64_t)t, ctr++);
                uint32_t r = (uint32_t)(word & 0xFFFFu);
                word >>= 16;
                int32_t ubit = (r >= tb), vbit = (r >= ta && r < tb) || (r >= tc);
                u = (u << 1) | ubit;
                v = (v << 1) | vbit;
            }
            if (u < nlimit && v < nlimit && u != v) break;
        }
        if (symmetric) {
            src[2 * t] = u;     dst[2 * t] = v;
            src[2 * t + 1] = v; dst[2 * t + 1] = u;
        } else {
            src[t] = u; dst[t] = v;
        }
    }
}

/* random relabelling of vertex ids: perm = Fisher-Yates shuffle of 0..n-1 */
void synth_relabel(int32_t n, int64_t E, uint64_t seed, int32_t* src, int32_t* dst) {
    int32_t* perm = (int32_t*)malloc((size_t)n * sizeof(int32_t));
    for (int32_t i = 0; i < n; ++i) perm[i] = i;
    for (int32_t i = n - 1; i > 0; --i) {
        int32_t j = (int32_t)ubelow(synth_u64(seed, 5, (uint64_t)i), (uint64_t)i + 1);
        int32_t t = perm[i]; perm[i] = perm[j]; perm[j] = t;
    }
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < E; ++k) { src[k] = perm[src[k]]; dst[k] = perm[dst[k]]; }
    free(perm);
}

/* reorder an edge list by target id, keeping the input order among equal targets
 * (the "sorted by dst" presentation of the largest workload).  Input generation only. */
void synth_sort_by_dst(int32_t n, int64_t E, int32_t* src, int32_t* dst) {
    int64_t* start = (int64_t*)calloc((size_t)n + 1, sizeof(int64_t));
    int32_t* s2 = (int32_t*)malloc((size_t)(E > 0 ? E : 1) * sizeof(int32_t));
    int32_t* d2 = (int32_t*)malloc((size_t)(E > 0 ? E : 1) * sizeof(int32_t));
    for (int64_t k = 0; k < E; ++k) start[dst[k] + 1]++;
    for (int32_t i = 0; i < n; ++i) start[i + 1] += start[i];
    for (int64_t k = 0; k < E; ++k) {
        int64_t p = start[dst[k]]++;
        s2[p] = src[k]; d2[p] = dst[k];
    }
    memcpy(src, s2, (size_t)E * sizeof(int32_t));
    memcpy(dst, d2, (size_t)E * sizeof(int32_t));
    free(start); free(s2); free(d2);
}
