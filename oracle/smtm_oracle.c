/*
 * CPU oracle for the SMTM semantic-memory hot path (arxiv 2112.02644).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * paper defines; the tests, the smoke check and the benchmark's CPU-baseline
 * leg call it.  The CUDA library never links, includes or calls it, and it
 * shares no code with the CUDA library.
 *
 * Everything floating point is computed in double, one frame at a time, in the
 * order the paper gives.  Integer state (frequency table, time-stamp table,
 * ranking, fast-memory size) is exact.  All pointers are host pointers and all
 * state lives in caller-owned arrays: the functions are stateless.
 *
 * Sections followed (equations numbered in order of appearance in the paper):
 *   Sec. 4.1            semantic vector = global average pooling      orc_gap
 *   Sec. 4.2  Eq. 1     cosine similarity                             orc_cosine
 *   Sec. 4.2  Eq. 2     single-layer separability                     orc_lookup_layer (sep)
 *   Sec. 5    Eq. 3     cross-layer cumulative similarity             orc_lookup_layer
 *   Sec. 5    Eq. 4     accumulated confidence and the exit rule      orc_lookup_layer
 *   Sec. 6.1            frequency table and time-stamp table          orc_tables_update
 *   Sec. 6.1  Eq. 5     replacement score and top-k                   orc_resize
 *   Sec. 6.2  Eq. 6     adaptive fast-memory size                     orc_resize
 *   Sec. 6.3  Eq. 7     running-mean semantic centres                 orc_centers_update
 *
 * Parity pins live in tests/test_oracle_*.py.  Unpinned: nothing in this file;
 * the paper's Table 1 and figures (dataset results) are "parity unpinned"
 * because the datasets, the models and the figures' numbers are not available.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_F32 = 0, ORC_F16 = 1, ORC_BF16 = 2 };
enum { ORC_NCHW = 0, ORC_NHWC = 1 };

/* ---- exact widening of the storage formats to double --------------------- */

static double widen_f32(const void* p, size_t i) {
    float f;
    memcpy(&f, (const char*)p + 4 * i, 4);
    return (double)f;
}

/* bfloat16 = the upper 16 bits of an IEEE binary32. */
static double widen_bf16(const void* p, size_t i) {
    uint16_t h;
    uint32_t u;
    float f;
    memcpy(&h, (const char*)p + 2 * i, 2);
    u = (uint32_t)h << 16;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static double widen_f16(const void* p, size_t i) {
    uint16_t h;
    int sign, ex, fr;
    double v;
    memcpy(&h, (const char*)p + 2 * i, 2);
    sign = (h >> 15) & 1;
    ex = (h >> 10) & 0x1f;
    fr = h & 0x3ff;
    if (ex == 0)
        v = ldexp((double)fr, -24); /* subnormal: fr * 2^-10 * 2^-14 */
    else if (ex == 31)
        v = fr ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)fr / 1024.0, ex - 15);
    return sign ? -v : v;
}

static double widen(const void* p, size_t i, int dtype) {
    if (dtype == ORC_F32) return widen_f32(p, i);
    if (dtype == ORC_F16) return widen_f16(p, i);
    return widen_bf16(p, i);
}

/* ---- Sec. 4.1: semantic vector ------------------------------------------- */

/* SV[b][c] = (1 / (H*W)) * sum over h, w of X[b][c][h][w]; frames with a
 * non-zero skip[b] are left untouched (skip may be NULL). */
int orc_gap(const void* x, int dtype, int layout, int B, int C, int H, int W,
            const uint8_t* skip, double* sv) {
    int b, c, h, w;
    if (dtype < 0 || dtype > 2 || layout < 0 || layout > 1) return 1;
    for (b = 0; b < B; ++b) {
        if (skip && skip[b]) continue;
        for (c = 0; c < C; ++c) {
            double sum = 0.0;
            for (h = 0; h < H; ++h)
                for (w = 0; w < W; ++w) {
                    size_t idx;
                    if (layout == ORC_NCHW)
                        idx = (((size_t)b * C + c) * H + h) * W + w;
                    else
                        idx = (((size_t)b * H + h) * W + w) * C + c;
                    sum += widen(x, idx, dtype);
                }
            sv[(size_t)b * C + c] = sum / ((double)H * (double)W);
        }
    }
    return 0;
}

/* ---- Sec. 4.2, Eq. 1: cosine similarity ----------------------------------- */

/* <a,b> / (|a| |b|); defined as 0 when either vector has zero length. */
double orc_cosine(const double* a, const double* b, int D) {
    double dot = 0.0, na = 0.0, nb = 0.0;
    int i;
    for (i = 0; i < D; ++i) {
        dot += a[i] * b[i];
        na += a[i] * a[i];
        nb += b[i] * b[i];
    }
    if (na == 0.0 || nb == 0.0) return 0.0;
    return dot / (sqrt(na) * sqrt(nb));
}

/* ---- top-1 / top-2 with the tie rule -------------------------------------- */

/* A NaN value ranks below everything.  Among equal values the lower class id
 * ranks first.  Returns the slots of the best and second best (-1 if absent). */
static int ranks_before(double va, int ida, double vb, int idb) {
    int na = isnan(va), nb = isnan(vb);
    if (na != nb) return nb; /* the non-NaN one ranks first */
    if (!na && va != vb) return va > vb;
    return ida < idb;
}

static void top2(const double* v, const int32_t* ids, int k, int* hi, int* sh) {
    int j;
    *hi = -1;
    *sh = -1;
    for (j = 0; j < k; ++j) {
        if (*hi < 0 || ranks_before(v[j], ids[j], v[*hi], ids[*hi])) {
            *sh = *hi;
            *hi = j;
        } else if (*sh < 0 || ranks_before(v[j], ids[j], v[*sh], ids[*sh])) {
            *sh = j;
        }
    }
}

/* (top - second) / second with the sign cases spelled out:
 *   top <= 0 (or NaN)           -> 0
 *   second NaN                  -> NaN (Eq. 2 / Eq. 4 as printed, on a NaN operand)
 *   second <= 0 < top           -> +inf
 *   otherwise                   -> Eq. 2 / Eq. 4 as printed. */
static double ratio_margin(double top, double second) {
    if (!(top > 0.0)) return 0.0;
    if (isnan(second)) return NAN;
    if (!(second > 0.0)) return INFINITY;
    return (top - second) / second;
}

/* ---- Sec. 5: lookup at one candidate exit layer --------------------------- */

/*
 * layer        1-based index l among the candidate exit layers.
 * sv           [B][D] semantic vectors of this layer (rows of done frames unused).
 * centers      [n][D] semantic centres SC_j^l of the global memory.
 * members      [S][k_max] class ids in fast memory, k[s] of them valid.
 * sa           [B][k_max] cumulative similarity per fast-memory slot (in/out).
 * force        NULL, or [B]: -1 = decide by the rule, 0 / 1 = decision imposed
 *              (used by the tests to follow a near-threshold decision).
 * Outputs for frames that are not done on entry: ac[b], sep[b], top[b][2]
 * (class ids, -1 if absent), and on exit done[b] = 1, exit_layer[b] = layer,
 * pred[b] = class of SA_H.  near[b] = 1 when |AC - tau| <= near_band.
 *
 * The decision is taken in single precision on the single-precision roundings
 * of SA_H and SA_SH, in division-free form:
 *     exit  <=>  SA_H > 0  and  SA_H - SA_SH > tau * max(SA_SH, 0)
 * which for SA_SH > 0 is Eq. 4's  AC > tau.  Fewer than two slots never exit.
 */
int orc_lookup_layer(int layer, int B, int D, const double* sv, const double* centers, int n,
                     const int32_t* stream_id, const int32_t* members, const int32_t* k,
                     int k_max, double tau, double near_band, double* sa, uint8_t* done,
                     int32_t* exit_layer, int32_t* pred, double* ac, double* sep,
                     int32_t* top, uint8_t* near, const int8_t* force) {
    int b, j;
    double weight = ldexp(1.0, layer - 1); /* weight_l = 2^(l-1), Sec. 5 */
    double* s = (double*)malloc(sizeof(double) * (size_t)(k_max > 0 ? k_max : 1));
    if (!s) return 2;
    for (b = 0; b < B; ++b) {
        int sid, kk, hi, sh, shi, ssh, leave;
        const int32_t* mem;
        double* sab;
        if (done[b]) continue;
        sid = stream_id ? stream_id[b] : 0;
        kk = k[sid];
        mem = members + (size_t)sid * k_max;
        sab = sa + (size_t)b * k_max;
        for (j = 0; j < kk; ++j) {
            int cls = mem[j];
            if (cls < 0 || cls >= n) {
                free(s);
                return 3;
            }
            s[j] = orc_cosine(sv + (size_t)b * D, centers + (size_t)cls * D, D); /* Eq. 1 */
            sab[j] += s[j] * weight;                                             /* Eq. 3 */
        }
        top2(sab, mem, kk, &hi, &sh);
        top2(s, mem, kk, &shi, &ssh);
        top[2 * b] = hi >= 0 ? mem[hi] : -1;
        top[2 * b + 1] = sh >= 0 ? mem[sh] : -1;
        if (sh < 0) { /* fewer than two entries: no second-highest, never exit */
            ac[b] = 0.0;
            sep[b] = 0.0;
            leave = 0;
        } else {
            float fh = (float)sab[hi], fs = (float)sab[sh], ft = (float)tau;
            float diff = fh - fs;
            float rhs = ft * (fs > 0.0f ? fs : 0.0f);
            ac[b] = ratio_margin(sab[hi], sab[sh]); /* Eq. 4 */
            sep[b] = ratio_margin(s[shi], s[ssh]);  /* Eq. 2 */
            leave = (fh > 0.0f) && (diff > rhs);
        }
        near[b] = (uint8_t)(isfinite(ac[b]) && fabs(ac[b] - tau) <= near_band);
        if (force && force[b] >= 0) leave = force[b] && hi >= 0;
        if (leave) {
            done[b] = 1;
            exit_layer[b] = layer;
            pred[b] = mem[hi];
        }
    }
    free(s);
    return 0;
}

/* ---- Sec. 6.1: frequency table and time-stamp table ----------------------- */

#define ORC_FT_MAX (1 << 20)

/* Frames in ascending index, each applied to the tables of its own stream:
 * the frame's class gets FT + 1 (saturating at 2^20) and TS = 0, every other
 * class of that stream gets TS + 1.  A frame whose label is -1 only ages. */
int orc_tables_update(int B, const int32_t* stream_id, const int32_t* final_label, int S, int n,
                      int32_t* ft, int32_t* ts) {
    int b, i;
    for (b = 0; b < B; ++b) {
        int sid = stream_id ? stream_id[b] : 0;
        int lab = final_label[b];
        int32_t* f = ft + (size_t)sid * n;
        int32_t* t = ts + (size_t)sid * n;
        if (sid < 0 || sid >= S || lab >= n) return 3;
        for (i = 0; i < n; ++i) {
            if (i == lab) {
                if (f[i] < ORC_FT_MAX) f[i] += 1;
                t[i] = 0;
            } else if (t[i] < INT32_MAX) {
                t[i] += 1;
            }
        }
    }
    return 0;
}

/* The variant of Sec. 7.1 ("decay the historical memory in the frequency table
 * based on the forgetting mechanism" of Sec. 6.1): the decay of Eq. 5 is applied
 * to the table itself.  FT is held in fixed point with ORC_FT_FRAC fractional
 * bits: an appearance adds one unit, and each time a class has gone another W
 * consecutive frames unseen (TS reaches a multiple of W) its FT is multiplied
 * by 0.25, rounding down.  Until the class reappears this keeps FT equal to
 * Eq. 5's score of the plain tables (up to that rounding), but the history
 * stays forgotten when it does reappear. */
#define ORC_FT_FRAC 10

int orc_tables_update_forgetting(int B, const int32_t* stream_id, const int32_t* final_label, int S, int n,
                                 int W, int32_t* ft, int32_t* ts) {
    int b, i;
    if (W < 1) return 1;
    for (b = 0; b < B; ++b) {
        int sid = stream_id ? stream_id[b] : 0;
        int lab = final_label[b];
        int32_t* f = ft + (size_t)sid * n;
        int32_t* t = ts + (size_t)sid * n;
        if (sid < 0 || sid >= S || lab >= n) return 3;
        for (i = 0; i < n; ++i) {
            if (i == lab) {
                int64_t v = (int64_t)f[i] + (1 << ORC_FT_FRAC);
                int64_t cap = (int64_t)ORC_FT_MAX << ORC_FT_FRAC;
                f[i] = (int32_t)(v > cap ? cap : v);
                t[i] = 0;
            } else if (t[i] < INT32_MAX) {
                t[i] += 1;
                if (t[i] % W == 0) f[i] >>= 2;
            }
        }
    }
    return 0;
}

/* ---- Sec. 6.3, Eq. 7: adaptive semantic centres --------------------------- */

/* For one layer l0 (1-based): every frame, in ascending index, whose final
 * label is j >= 0 and whose inference stopped at a layer >= l0 moves centre j:
 *     SC' = (SC * m + SV) / (m + 1),   m' = m + 1. */
int orc_centers_update(int l0, int B, int D, const double* sv, const int32_t* final_label,
                       const int32_t* stop_layer, int n, double* centers, uint32_t* m) {
    int b, d;
    for (b = 0; b < B; ++b) {
        int j = final_label[b];
        double* sc;
        double mm;
        if (j < 0 || stop_layer[b] < l0) continue;
        if (j >= n) return 3;
        sc = centers + (size_t)j * D;
        mm = (double)m[j];
        for (d = 0; d < D; ++d) sc[d] = (sc[d] * mm + sv[(size_t)b * D + d]) / (mm + 1.0);
        m[j] += 1;
    }
    return 0;
}

/* ---- Sec. 6.1 Eq. 5 and Sec. 6.2 Eq. 6: replacement and adaptive size ------ */

#define ORC_E_MAX 12

/* Score_i = FT_i * 0.25^floor(TS_i / W), held exactly as the integer
 * FT_i * 4^(12 - e_i) with e_i = min(floor(TS_i / W), 12). */
uint64_t orc_score(int32_t ft, int32_t ts, int W) {
    int e = ts / W;
    uint64_t f = (uint64_t)(ft < 0 ? 0 : (ft > ORC_FT_MAX ? ORC_FT_MAX : ft));
    if (e > ORC_E_MAX) e = ORC_E_MAX;
    return f << (2 * (ORC_E_MAX - e));
}

/* Per stream: rank all n classes by (score descending, class id ascending);
 * the fast-memory size becomes the smallest k in [k_min, k_max] with
 *     sum of the k best scores / sum of all scores  >  cl_num / cl_den
 * (k_max when none does), and the fast memory the first k of the ranking
 * (members holds the first k_max of it).  A stream whose scores are all zero
 * keeps its size and members.  forgetting != 0: the tables are those of
 * orc_tables_update_forgetting. */
int orc_resize(int S, int n, const int32_t* ft, const int32_t* ts, int W, int k_min, int k_max,
               int cl_num, int cl_den, int forgetting, int32_t* members, int32_t* k) {
    int s, i, j;
    uint64_t* score;
    int32_t* order;
    if (n < 1 || k_max > n || k_min < 1 || k_min > k_max || W < 1) return 1;
    score = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)n);
    order = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    if (!score || !order) {
        free(score);
        free(order);
        return 2;
    }
    for (s = 0; s < S; ++s) {
        uint64_t total = 0, prefix = 0;
        int chosen = k_max;
        for (i = 0; i < n; ++i) {
            /* with the forgetting tables the decay already sits in FT: the score is FT itself */
            score[i] = forgetting ? (uint64_t)(ft[(size_t)s * n + i] < 0 ? 0 : ft[(size_t)s * n + i])
                                  : orc_score(ft[(size_t)s * n + i], ts[(size_t)s * n + i], W);
            total += score[i];
        }
        if (total == 0) continue;
        /* insertion sort, stable: equal scores stay in ascending class id */
        for (i = 0; i < n; ++i) {
            j = i;
            while (j > 0 && score[order[j - 1]] < score[i]) {
                order[j] = order[j - 1];
                --j;
            }
            order[j] = i;
        }
        for (i = 0; i < k_max; ++i) {
            prefix += score[order[i]];
            if (i + 1 >= k_min && (uint64_t)cl_den * prefix > (uint64_t)cl_num * total) {
                chosen = i + 1;
                break;
            }
        }
        for (i = 0; i < k_max; ++i) members[(size_t)s * k_max + i] = order[i];
        k[s] = chosen;
    }
    free(score);
    free(order);
    return 0;
}
