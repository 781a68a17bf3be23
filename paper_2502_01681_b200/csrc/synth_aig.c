/*
 * Seeded synthetic And-Inverter-Graph generators (host only, plain C).
 *
 * This file only draws random circuits: node ids in topological order, fan-in
 * lists as a destination-sorted CSR and the logic level of every node.  It holds
 * no attention / projection / graph-prep arithmetic; it is the one piece of code
 * that both the CPU checker and the CUDA library are fed from.
 *
 * Circuit shapes follow the dataset statistics the paper tabulates (three node
 * kinds told apart by in-degree 0 / 1 / 2, fewer than two edges per node, a few
 * per cent primary inputs, depth from tens to thousands of levels).
 *
 * Randomness: a counter-based generator, splitmix64 applied to
 * (seed, stream, index), so any element can be drawn independently.
 */
#include <stdint.h>
#include <stddef.h>
#include <math.h>

static inline uint64_t splitmix64(uint64_t x) {
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

/* uniform double in [0,1) from (seed, stream, index) */
static inline double u01(uint64_t seed, uint64_t stream, uint64_t index) {
    uint64_t k = splitmix64(seed ^ splitmix64(stream * 0xD1B54A32D192ED03ull + 0x632BE59BD9B4E019ull));
    uint64_t r = splitmix64(k + index * 0x9E3779B97F4A7C15ull);
    return (double)(r >> 11) * (1.0 / 9007199254740992.0);
}

enum { STREAM_KIND = 1, STREAM_WIN = 2, STREAM_FAN0 = 3, STREAM_FAN1 = 4 };

/*
 * Window generator.  Nodes 0..n_pi-1 are primary inputs; gate i (id order is a
 * topological order) is a NOT with probability not_ratio, else an AND.  Its
 * fan-ins are drawn uniformly, without replacement, from the previous
 * min(W_i, i) nodes, where W_i = win_fixed if win_fixed > 0, else
 * floor(2^U), U ~ Uniform[win_lo_exp, win_hi_exp).
 *
 * Outputs: row_ptr[n+1], col_idx[<= 2*n_gates] (sources ascending within a
 * row), level[n] (0 for a primary input, else 1 + max over fan-ins).
 * Returns the number of edges, or -1 on bad arguments.
 */
int64_t dg4_synth_window_aig(uint64_t seed, int32_t n_pi, int32_t n_gates,
                             int32_t win_fixed, double win_lo_exp, double win_hi_exp,
                             double not_ratio,
                             int32_t* row_ptr, int32_t* col_idx, int32_t* level) {
    if (n_pi < 2 || n_gates < 0 || !row_ptr || !col_idx || !level) return -1;
    int64_t n = (int64_t)n_pi + n_gates;
    int64_t e = 0;
    for (int32_t i = 0; i < n_pi; ++i) { row_ptr[i] = 0; level[i] = 0; }
    for (int64_t i = n_pi; i < n; ++i) {
        row_ptr[i] = (int32_t)e;
        int64_t w;
        if (win_fixed > 0) {
            w = win_fixed;
        } else {
            double u = win_lo_exp + (win_hi_exp - win_lo_exp) * u01(seed, STREAM_WIN, (uint64_t)i);
            w = (int64_t)floor(exp2(u));
        }
        if (w > i) w = i;
        if (w < 2) w = 2;
        int is_not = u01(seed, STREAM_KIND, (uint64_t)i) < not_ratio;
        int64_t off0 = (int64_t)(u01(seed, STREAM_FAN0, (uint64_t)i) * (double)w);
        if (off0 >= w) off0 = w - 1;
        int64_t a = i - 1 - off0;
        if (is_not) {
            col_idx[e++] = (int32_t)a;
            level[i] = level[a] + 1;
        } else {
            int64_t off1 = (int64_t)(u01(seed, STREAM_FAN1, (uint64_t)i) * (double)(w - 1));
            if (off1 >= w - 1) off1 = w - 2;
            if (off1 >= off0) off1 += 1;           /* skip the slot already taken */
            int64_t b = i - 1 - off1;
            int64_t lo = a < b ? a : b, hi = a < b ? b : a;
            col_idx[e++] = (int32_t)lo;
            col_idx[e++] = (int32_t)hi;
            int32_t la = level[a], lb = level[b];
            level[i] = (la > lb ? la : lb) + 1;
        }
    }
    row_ptr[n] = (int32_t)e;
    return e;
}

/*
 * Layered generator.  n_pi primary inputs form level 0; then n_levels levels of
 * gates_per_level gates each, ids assigned level by level.  A gate on level l
 * takes its first fan-in uniformly from level l-1 and, if it is an AND, its
 * second one uniformly from levels max(0, l-3) .. l-1, distinct from the first.
 * So every gate's level equals its layer index exactly.
 */
int64_t dg4_synth_layered_aig(uint64_t seed, int32_t n_pi, int32_t n_levels, int32_t gates_per_level,
                              double not_ratio,
                              int32_t* row_ptr, int32_t* col_idx, int32_t* level) {
    if (n_pi < 2 || n_levels < 0 || gates_per_level < 2 || !row_ptr || !col_idx || !level) return -1;
    int64_t n = (int64_t)n_pi + (int64_t)n_levels * gates_per_level;
    int64_t e = 0;
    for (int32_t i = 0; i < n_pi; ++i) { row_ptr[i] = 0; level[i] = 0; }
    for (int32_t l = 1; l <= n_levels; ++l) {
        /* id range of level l-1 and of levels max(0,l-3)..l-1 */
        int64_t prev_begin = (l == 1) ? 0 : (int64_t)n_pi + (int64_t)(l - 2) * gates_per_level;
        int64_t prev_end   = (int64_t)n_pi + (int64_t)(l - 1) * gates_per_level;
        int32_t l3 = l - 3 < 0 ? 0 : l - 3;
        int64_t span_begin = (l3 == 0) ? 0 : (int64_t)n_pi + (int64_t)(l3 - 1) * gates_per_level;
        int64_t span = prev_end - span_begin;
        for (int32_t g = 0; g < gates_per_level; ++g) {
            int64_t i = prev_end + g;
            row_ptr[i] = (int32_t)e;
            level[i] = l;
            int64_t pw = prev_end - prev_begin;
            int64_t a = prev_begin + (int64_t)(u01(seed, STREAM_FAN0, (uint64_t)i) * (double)pw);
            if (a >= prev_end) a = prev_end - 1;
            int is_not = u01(seed, STREAM_KIND, (uint64_t)i) < not_ratio;
            if (is_not) {
                col_idx[e++] = (int32_t)a;
            } else {
                int64_t r = (int64_t)(u01(seed, STREAM_FAN1, (uint64_t)i) * (double)(span - 1));
                if (r >= span - 1) r = span - 2;
                int64_t b = span_begin + r;
                if (b >= a) b += 1;
                int64_t lo = a < b ? a : b, hi = a < b ? b : a;
                col_idx[e++] = (int32_t)lo;
                col_idx[e++] = (int32_t)hi;
            }
        }
    }
    row_ptr[n] = (int32_t)e;
    return e;
}
