/*
 * ecco_oracle.c -- plain, slow, single-threaded CPU oracle of the Ecco 4x block codec.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the checker the CUDA library is compared with.
 * It shares no code, header, table or constant generator with the library; only the tests,
 * the smoke check and the benchmark's cpu_baseline / reference arm may call it.
 *
 * What it implements, in the paper's order and notation (Ecco, Sec. 3.2 "Model Compression",
 * Sec. 4.2 "Decompressor Design", Sec. 4.3 "Compressor Design"):
 *
 *   Step 1  partition into groups of 128                       (Sec. 3.2, Fig. 4 step 1)
 *   Step 2  two-level normalisation: group abs-max -> FP8 under a per-tensor power-of-two
 *           FP16-to-FP8 factor T = 2^e; values / scale          (Fig. 4 step 2)
 *   Step 3  per-group k-means, 15 clusters on the 127 other values (Fig. 4 step 3)
 *   Step 4  k-means with S clusters over the group patterns     (Fig. 4 step 4)
 *   Step 5  round to every shared pattern, keep the min-MSE one (Fig. 4 step 5), or the
 *           min/max fitness rule of the KV path                 (Sec. 3.2 "KV Cache Compression",
 *                                                                Sec. 4.3 pattern selector)
 *   Step 6  k-means with H clusters over index histograms       (Fig. 4 step 6)
 *   Step 7  histograms -> Huffman codebooks, lengths 2..8       (Fig. 4 step 7, Sec. 4.2)
 *   Step 8  per group, the codebook giving the shortest stream  (Fig. 4 step 8)
 *   Step 9  clip, or pad with 15-bit outliers, to 64 bytes      (Fig. 4 step 9)
 *   Decoder: pattern retriever, Huffman decode, outlier count, mapper (Sec. 4.2)
 *   Consumers: decode-phase GEMV and attention scores QK^T/sqrt(d) (Sec. 2.1) in fp64.
 *
 * Where the paper is silent (bit order inside the block, FP8 flavour, tie rules, pad cap)
 * a reading had to be chosen; each is marked "reading:" where it is used below.
 *
 * Pins (tests/test_oracle_*.py): FP16/FP8 conversion against numpy / torch exhaustively;
 * exact dequantisation; DP k-means against brute force; Kraft equality, prefix-freeness,
 * textbook-Huffman cost and entropy bound for every code; package-merge against brute
 * force; brute-force pattern choice; encode->decode round trip; hand-assembled golden block.
 * Parity unpinned: the Lloyd iterations of steps 4 and 6 (heuristic; only monotonicity and
 * determinism are checked), the optional activation weights of step 3, the block bit order
 * and the cap of 16 pads (both are this build's definitions, self-consistency only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define EO_G 128         /* values per group (Sec. 3.1 "Target Compression Ratio") */
#define EO_BLOCK 64      /* bytes per compressed block (Sec. 3.1 "Target Compressed Block Size") */
#define EO_BITS 512
#define EO_NC 15         /* centroids per pattern (Sec. 3.2) */
#define EO_NSYM 16       /* 15 centroid indices + index 15 for the abs-max (Sec. 3.2) */
#define EO_MAXS 64
#define EO_H 4
#define EO_PAD_BITS 15   /* 7-bit location + 8-bit FP8 value (Sec. 3.2) */
#define EO_MAX_PADS 16   /* reading: the sorter's "top 16" (Sec. 4.3) caps the pads */
#define EO_KP_MAXLEN 12  /* reading: the paper gives no limit for the ID_KP code */

#define EO_SELECT_MSE 0
#define EO_SELECT_MINMAX 1

#define EO_OK 0
#define EO_ERR_ARG (-1)
#define EO_ERR_NONFINITE (-3)
#define EO_ERR_META (-4)

typedef struct {
    int32_t S;                            /* number of shared patterns, 2..64 */
    int32_t H;                            /* codebooks per pattern, fixed 4 */
    int32_t e;                            /* per-tensor FP16-to-FP8 factor T = 2^e */
    int32_t reserved;
    uint16_t pattern[EO_MAXS][16];        /* fp16 bits, ascending; entry 15 unused (0) */
    uint8_t cb_len[EO_MAXS][EO_H][EO_NSYM]; /* code lengths, 2..8 */
    uint8_t kp_len[EO_MAXS];              /* ID_KP code lengths, 1..12 */
} eo_meta;

typedef struct {
    uint64_t n_groups;
    uint64_t clipped_groups;   /* groups that lost at least one value */
    uint64_t clipped_values;
    uint64_t padded_groups;
    uint64_t padded_values;
    uint64_t total_bits;       /* header + codewords actually stored, before pads */
    uint64_t kp_usage[EO_MAXS];
    uint64_t hf_usage[EO_H];
    uint64_t sym_count[EO_NSYM];
} eo_stats;

/* ------------------------------------------------------------------------------------ */
/* Number formats.                                                                       */
/* ------------------------------------------------------------------------------------ */

/* IEEE binary16 -> binary32, from the definition of the format. */
float eo_fp16_to_f32(uint16_t h)
{
    int sign = (h >> 15) & 1, E = (h >> 10) & 31, m = h & 1023;
    double v;
    if (E == 31) v = m ? NAN : INFINITY;
    else if (E == 0) v = ldexp((double)m, -24);
    else v = ldexp(1.0 + m / 1024.0, E - 15);
    return (float)(sign ? -v : v);
}

/* binary32 -> binary16, round to nearest, ties to even, from the definition. */
uint16_t eo_f32_to_fp16(float f)
{
    uint16_t sign = signbit(f) ? 0x8000u : 0;
    double v = fabs((double)f);
    if (isnan(f)) return (uint16_t)(sign | 0x7e00u);
    if (v >= 65520.0) return (uint16_t)(sign | 0x7c00u); /* 65520 is the tie that rounds up to 2^16 */
    if (v < ldexp(1.0, -14)) {
        /* subnormal grid of 2^-24; rint is ties-to-even in the default rounding mode;
           a result of 1024 is the smallest normal, whose bit pattern is also 1024 */
        return (uint16_t)(sign | (uint16_t)rint(ldexp(v, 24)));
    }
    int ex;
    (void)frexp(v, &ex);       /* v = m * 2^ex, m in [0.5, 1) */
    int E = ex - 1;            /* v = 1.xxx * 2^E */
    long q = (long)rint(ldexp(v, 10 - E)); /* in [1024, 2048] */
    if (q == 2048) { q = 1024; E += 1; }
    return (uint16_t)(sign | ((E + 15) << 10) | (q - 1024));
}

/* reading: "FP8" is OCP E4M3 (1-4-3, bias 7, largest finite 448, no infinity).  The decoder is
   purely arithmetic, so the byte S.1111.111 (a NaN in OCP) reads as 480; the encoder never
   writes it, and a corrupt block then still decodes to a number. */
float eo_e4m3_to_f32(uint8_t b)
{
    int sign = b >> 7, E = (b >> 3) & 15, m = b & 7;
    double v = (E == 0) ? ldexp((double)m, -9) : ldexp(1.0 + m / 8.0, E - 7);
    return (float)(sign ? -v : v);
}

/* binary32 -> E4M3, round to nearest even, saturating at +-448. */
uint8_t eo_e4m3_from_f32(float f)
{
    uint8_t sign = signbit(f) ? 0x80u : 0;
    double v = fabs((double)f);
    if (isnan(f)) return (uint8_t)(sign | 0x7e);
    if (v >= 448.0) return (uint8_t)(sign | 0x7e);
    if (v < ldexp(1.0, -6)) return (uint8_t)(sign | (uint8_t)rint(ldexp(v, 9)));
    int ex;
    (void)frexp(v, &ex);
    int E = ex - 1;
    long q = (long)rint(ldexp(v, 3 - E)); /* in [8, 16] */
    if (q == 16) { q = 8; E += 1; }
    int bits = ((E + 7) << 3) | (int)(q - 8);
    if (bits > 0x7e) bits = 0x7e;
    return (uint8_t)(sign | bits);
}

/* ------------------------------------------------------------------------------------ */
/* Canonical prefix codes.                                                               */
/* ------------------------------------------------------------------------------------ */

/* Canonical code from lengths: symbols ordered by (length, symbol id); the first gets the
   all-zero code, each next one the previous code plus one, shifted left when the length
   grows.  A length of 0 means the symbol has no code.  Returns the Kraft sum numerator
   over 2^maxlen through *kraft_num (so a complete code has *kraft_num == 2^maxlen). */
void eo_canonical_codes(const uint8_t* len, int n, int maxlen, uint16_t* code, uint32_t* kraft_num)
{
    uint32_t next = 0, kraft = 0;
    int prev_len = 0;
    for (int L = 1; L <= maxlen; ++L)
        for (int s = 0; s < n; ++s)
            if (len[s] == L) {
                if (prev_len) next = (next + 1) << (L - prev_len);
                code[s] = (uint16_t)next;
                prev_len = L;
                kraft += 1u << (maxlen - L);
            }
    if (kraft_num) *kraft_num = kraft;
}

/* Step 7: optimal prefix code over all 16 symbols with every length in [2, 8] (Sec. 4.2:
   "limiting the code length to 2-8 bits") and Kraft sum exactly 1.
   reading: exhaustive search over the number of codes of each length (n2..n8); for a fixed
   multiset of lengths the cheapest assignment gives the shortest codes to the most frequent
   symbols (ties: lower symbol id first).  Among equal costs the first vector in
   lexicographic order of (n2, n3, ..., n8) wins. */
typedef struct { const double* sorted; double best; int bestn[9]; int n[9]; } eo_enum;

/* enumerate n[L..8] given `left` symbols and `kraft_left` (in units of 2^-8) still to place */
static void eo_enum_lengths(eo_enum* E, int L, int left, int kraft_left)
{
    if (L == 8) {
        if (left != kraft_left) return;          /* every 8-bit code is worth 2^-8 */
        E->n[8] = left;
        double cost = 0.0;
        int r = 0;
        for (int l = 2; l <= 8; ++l)
            for (int c = 0; c < E->n[l]; ++c) cost += E->sorted[r++] * l;
        if (cost < E->best) { E->best = cost; memcpy(E->bestn, E->n, sizeof E->n); }
        return;
    }
    int worth = 1 << (8 - L);
    for (int c = 0; c <= left && c * worth <= kraft_left; ++c) {
        E->n[L] = c;
        eo_enum_lengths(E, L + 1, left - c, kraft_left - c * worth);
    }
}

int eo_huffman_2_8(const double* freq, uint8_t* len)
{
    int order[EO_NSYM];
    double sorted[EO_NSYM];
    for (int i = 0; i < EO_NSYM; ++i) order[i] = i;
    for (int i = 1; i < EO_NSYM; ++i) {          /* stable insertion sort, descending freq */
        int s = order[i], j = i;
        while (j > 0 && freq[order[j - 1]] < freq[s]) { order[j] = order[j - 1]; --j; }
        order[j] = s;
    }
    for (int i = 0; i < EO_NSYM; ++i) {
        if (!(freq[order[i]] >= 0.0)) return EO_ERR_ARG;
        sorted[i] = freq[order[i]];
    }
    eo_enum E;
    memset(&E, 0, sizeof E);
    E.sorted = sorted; E.best = INFINITY;
    eo_enum_lengths(&E, 2, EO_NSYM, 256);
    if (!(E.best < INFINITY)) return EO_ERR_ARG;
    int r = 0;
    for (int L = 2; L <= 8; ++L)
        for (int c = 0; c < E.bestn[L]; ++c) len[order[r++]] = (uint8_t)L;
    return EO_OK;
}

/* Length-limited optimal prefix code by the package-merge algorithm (Larmore & Hirschberg):
   every symbol is a coin of each denomination 2^-1 .. 2^-maxlen with its weight as the cost;
   the cheapest set of coins worth n-1 gives the lengths (length = coins bought of that
   symbol).  Used for the ID_KP code (reading: built from pattern usage + 1, at most 12 bits).
   Requires 2 <= n <= 64 and 2^maxlen >= n. */
typedef struct { double w; uint8_t cnt[EO_MAXS]; } eo_pkg;

static int eo_pkg_cmp(const void* a, const void* b)
{
    double x = ((const eo_pkg*)a)->w, y = ((const eo_pkg*)b)->w;
    return (x > y) - (x < y);
}

int eo_huffman_limited(const double* freq, int n, int maxlen, uint8_t* len)
{
    if (n < 2 || n > EO_MAXS || maxlen < 1 || maxlen > 16 || (1 << maxlen) < n) return EO_ERR_ARG;
    eo_pkg* leaves = (eo_pkg*)calloc((size_t)n, sizeof(eo_pkg));
    eo_pkg* cur = (eo_pkg*)calloc((size_t)(2 * n), sizeof(eo_pkg));
    eo_pkg* nxt = (eo_pkg*)calloc((size_t)(2 * n), sizeof(eo_pkg));
    if (!leaves || !cur || !nxt) { free(leaves); free(cur); free(nxt); return EO_ERR_ARG; }
    for (int s = 0; s < n; ++s) { leaves[s].w = freq[s]; leaves[s].cnt[s] = 1; }
    /* stable order: sort by weight, ties by symbol id (qsort is not stable, so sort indices) */
    for (int i = 1; i < n; ++i) {
        eo_pkg t = leaves[i]; int j = i;
        while (j > 0 && leaves[j - 1].w > t.w) { leaves[j] = leaves[j - 1]; --j; }
        leaves[j] = t;
    }
    int ncur = n;
    memcpy(cur, leaves, (size_t)n * sizeof(eo_pkg));     /* denomination 2^-maxlen */
    for (int level = maxlen - 1; level >= 1; --level) {
        /* package pairs of the current list, merge with a fresh copy of the leaves */
        int np = ncur / 2, nn = 0;
        for (int p = 0; p < np; ++p) {
            eo_pkg q; q.w = cur[2 * p].w + cur[2 * p + 1].w;
            for (int s = 0; s < EO_MAXS; ++s) q.cnt[s] = (uint8_t)(cur[2 * p].cnt[s] + cur[2 * p + 1].cnt[s]);
            nxt[nn++] = q;
        }
        for (int s = 0; s < n; ++s) nxt[nn++] = leaves[s];
        /* merge: packages first so that on equal weight a package precedes a leaf; any fixed
           rule gives an optimal code */
        for (int i = 1; i < nn; ++i) {
            eo_pkg t = nxt[i]; int j = i;
            while (j > 0 && nxt[j - 1].w > t.w) { nxt[j] = nxt[j - 1]; --j; }
            nxt[j] = t;
        }
        eo_pkg* tmp = cur; cur = nxt; nxt = tmp; ncur = nn;
    }
    (void)eo_pkg_cmp;
    /* the first 2n-2 items of the denomination-1/2 list are worth n-1 */
    memset(len, 0, (size_t)n);
    for (int i = 0; i < 2 * n - 2; ++i)
        for (int s = 0; s < n; ++s) len[s] = (uint8_t)(len[s] + cur[i].cnt[s]);
    free(leaves); free(cur); free(nxt);
    return EO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Clustering.                                                                           */
/* ------------------------------------------------------------------------------------ */

/* Step 3: exact weighted 1-D k-means by dynamic programming over the sorted values.
   v must be sorted ascending; w >= 0 (NULL = all ones).  Splits v into exactly k non-empty
   contiguous runs minimising the weighted sum of squared distances to the run means;
   ties take the earliest split.  Writes the k means (ascending) and returns the optimum.
   reading: "activation-aware" = optional per-element weights; k-means solved exactly so
   that no seed or iteration count is involved. */
double eo_kmeans1d(const double* v, const double* w, int n, int k, double* centroid)
{
    if (n < k || k < 1) return -1.0;
    double* pw = (double*)calloc((size_t)n + 1, sizeof(double));
    double* pwv = (double*)calloc((size_t)n + 1, sizeof(double));
    double* pwvv = (double*)calloc((size_t)n + 1, sizeof(double));
    double* D = (double*)malloc(sizeof(double) * (size_t)(k + 1) * (size_t)(n + 1));
    int* B = (int*)malloc(sizeof(int) * (size_t)(k + 1) * (size_t)(n + 1));
    for (int i = 0; i < n; ++i) {
        double wi = w ? w[i] : 1.0;
        pw[i + 1] = pw[i] + wi;
        pwv[i + 1] = pwv[i] + wi * v[i];
        pwvv[i + 1] = pwvv[i] + wi * v[i] * v[i];
    }
#define EO_COST(i, j) /* run v[i..j-1] */ \
    ((pw[j] - pw[i]) > 0.0 ? fmax(0.0, (pwvv[j] - pwvv[i]) - (pwv[j] - pwv[i]) * (pwv[j] - pwv[i]) / (pw[j] - pw[i])) : 0.0)
    for (int m = 0; m <= k; ++m)
        for (int j = 0; j <= n; ++j) { D[m * (n + 1) + j] = INFINITY; B[m * (n + 1) + j] = -1; }
    D[0] = 0.0;
    for (int m = 1; m <= k; ++m)
        for (int j = m; j <= n; ++j)
            for (int i = m - 1; i < j; ++i) {
                double prev = D[(m - 1) * (n + 1) + i];
                if (prev == INFINITY) continue;
                double c = prev + EO_COST(i, j);
                if (c < D[m * (n + 1) + j]) { D[m * (n + 1) + j] = c; B[m * (n + 1) + j] = i; }
            }
    double opt = D[k * (n + 1) + n];
    int j = n;
    for (int m = k; m >= 1; --m) {
        int i = B[m * (n + 1) + j];
        double sw = pw[j] - pw[i];
        if (sw > 0.0) centroid[m - 1] = (pwv[j] - pwv[i]) / sw;
        else { double s = 0.0; for (int t = i; t < j; ++t) s += v[t]; centroid[m - 1] = s / (j - i); }
        j = i;
    }
#undef EO_COST
    free(pw); free(pwv); free(pwvv); free(D); free(B);
    return opt;
}

/* splitmix64: the oracle's own counter-based generator for the seeded initialisations. */
static uint64_t eo_splitmix(uint64_t* state)
{
    uint64_t z = (*state += 0x9e3779b97f4a7c15ull);
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ull;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebull;
    return z ^ (z >> 31);
}
static double eo_uniform(uint64_t* state) { return (double)(eo_splitmix(state) >> 11) * (1.0 / 9007199254740992.0); }

static double eo_sqdist(const double* a, const double* b, int d)
{
    double s = 0.0;
    for (int i = 0; i < d; ++i) s += (a[i] - b[i]) * (a[i] - b[i]);
    return s;
}

/* Steps 4 and 6: Lloyd's k-means on n points of dimension d.
   reading: k-means++ seeding from a 64-bit seed, at most max_iter rounds, nearest-centre
   ties to the lower index, an empty cluster is re-seeded at the point farthest from its
   centre.  Writes centres [k][d], assignments [n], and (if obj_trace != NULL) the objective
   after every assignment step (max_iter + 1 entries, unused ones set to -1).
   Returns the number of rounds done. */
int eo_lloyd(const double* x, int n, int d, int k, uint64_t seed, int max_iter,
             double* centre, int32_t* assign, double* obj_trace)
{
    uint64_t st = seed;
    double* mind = (double*)malloc(sizeof(double) * (size_t)n);
    /* k-means++ */
    int first = (int)(eo_uniform(&st) * n); if (first >= n) first = n - 1;
    memcpy(centre, x + (size_t)first * d, sizeof(double) * (size_t)d);
    for (int i = 0; i < n; ++i) mind[i] = eo_sqdist(x + (size_t)i * d, centre, d);
    for (int c = 1; c < k; ++c) {
        double tot = 0.0;
        for (int i = 0; i < n; ++i) tot += mind[i];
        int pick = n - 1;
        if (tot > 0.0) {
            double r = eo_uniform(&st) * tot, acc = 0.0;
            for (int i = 0; i < n; ++i) { acc += mind[i]; if (acc > r) { pick = i; break; } }
        } else {
            pick = (int)(eo_uniform(&st) * n); if (pick >= n) pick = n - 1;
        }
        memcpy(centre + (size_t)c * d, x + (size_t)pick * d, sizeof(double) * (size_t)d);
        for (int i = 0; i < n; ++i) {
            double dd = eo_sqdist(x + (size_t)i * d, centre + (size_t)c * d, d);
            if (dd < mind[i]) mind[i] = dd;
        }
    }
    if (obj_trace) for (int t = 0; t <= max_iter; ++t) obj_trace[t] = -1.0;
    for (int i = 0; i < n; ++i) assign[i] = -1;
    double* sum = (double*)malloc(sizeof(double) * (size_t)k * (size_t)d);
    int* cnt = (int*)malloc(sizeof(int) * (size_t)k);
    int it = 0;
    for (;;) {
        int changed = 0;
        double obj = 0.0;
        for (int i = 0; i < n; ++i) {
            int best = 0; double bd = INFINITY;
            for (int c = 0; c < k; ++c) {
                double dd = eo_sqdist(x + (size_t)i * d, centre + (size_t)c * d, d);
                if (dd < bd) { bd = dd; best = c; }
            }
            if (assign[i] != best) { assign[i] = best; changed = 1; }
            mind[i] = bd; obj += bd;
        }
        if (obj_trace) obj_trace[it] = obj;
        if (!changed || it == max_iter) break;
        ++it;
        memset(sum, 0, sizeof(double) * (size_t)k * (size_t)d);
        memset(cnt, 0, sizeof(int) * (size_t)k);
        for (int i = 0; i < n; ++i) {
            cnt[assign[i]]++;
            for (int j = 0; j < d; ++j) sum[(size_t)assign[i] * d + j] += x[(size_t)i * d + j];
        }
        for (int c = 0; c < k; ++c) {
            if (cnt[c] > 0) {
                for (int j = 0; j < d; ++j) centre[(size_t)c * d + j] = sum[(size_t)c * d + j] / cnt[c];
            } else {
                int far = 0;
                for (int i = 1; i < n; ++i) if (mind[i] > mind[far]) far = i;
                memcpy(centre + (size_t)c * d, x + (size_t)far * d, sizeof(double) * (size_t)d);
                mind[far] = 0.0;
            }
        }
    }
    free(mind); free(sum); free(cnt);
    return it;
}

/* ------------------------------------------------------------------------------------ */
/* Per-group quantisation (Fig. 4 steps 2 and 5).                                        */
/* ------------------------------------------------------------------------------------ */

/* Per-tensor FP16-to-FP8 factor.  reading: T = 2^e with the smallest e in [-32, 16] such
   that max|x| <= 448 * 2^e (so the largest group scale does not saturate). */
int eo_choose_exponent(const uint16_t* x, uint64_t n, int32_t* e_out)
{
    double mx = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        float f = eo_fp16_to_f32(x[i]);
        if (!isfinite(f)) return EO_ERR_NONFINITE;
        if (fabs((double)f) > mx) mx = fabs((double)f);
    }
    int e = -32;
    while (e < 16 && mx > 448.0 * ldexp(1.0, e)) ++e;
    *e_out = e;
    return EO_OK;
}

/* index of the centroid nearest to u; ties to the lower index */
static int eo_nearest(const float* c, float u)
{
    int best = 0; double bd = INFINITY;
    for (int j = 0; j < EO_NC; ++j) {
        double d = ((double)u - (double)c[j]) * ((double)u - (double)c[j]);
        if (d < bd) { bd = d; best = j; }
    }
    return best;
}

/* Steps 2 and 5 for one group.  Outputs: position p* of the abs-max (first on ties), its
   signed FP8 byte q_s, the normalised values u[128] (u[p*] unused = 0), the chosen pattern
   and the 128 symbols (symbol 15 at p*).
   reading: the FP8 byte keeps the sign of the abs-max element so that index 15 restores it;
   the other values are divided by the *rounded* scale; a zero scale makes every u zero. */
int eo_quantize_group(const eo_meta* M, const uint16_t* x16, int select, int32_t* pstar_out,
                      uint8_t* qs_out, float* u, int32_t* kp_out, uint8_t* sym, double* err_out)
{
    float x[EO_G];
    float T = (float)ldexp(1.0, M->e);
    int p = 0;
    for (int i = 0; i < EO_G; ++i) {
        x[i] = eo_fp16_to_f32(x16[i]);
        if (!isfinite(x[i])) return EO_ERR_NONFINITE;
        if (fabsf(x[i]) > fabsf(x[p])) p = i;
    }
    uint8_t qs = eo_e4m3_from_f32(x[p] / T);
    float s = fabsf(eo_e4m3_to_f32(qs)) * T;
    for (int i = 0; i < EO_G; ++i) u[i] = (i == p || s == 0.0f) ? 0.0f : x[i] / s;

    int best = 0; double best_score = INFINITY;
    for (int k = 0; k < M->S; ++k) {
        float c[EO_NC];
        for (int j = 0; j < EO_NC; ++j) c[j] = eo_fp16_to_f32(M->pattern[k][j]);
        double score = 0.0;
        if (select == EO_SELECT_MSE) {
            /* Fig. 4 step 5: squared error after rounding to pattern k, abs-max excluded */
            for (int i = 0; i < EO_G; ++i) {
                if (i == p) continue;
                double d = (double)u[i] - (double)c[eo_nearest(c, u[i])];
                score += d * d;
            }
        } else {
            /* Sec. 4.3: squared difference of the group's min/max and the pattern's min/max */
            double lo = INFINITY, hi = -INFINITY;
            for (int i = 0; i < EO_G; ++i) {
                if (i == p) continue;
                if (u[i] < lo) lo = u[i];
                if (u[i] > hi) hi = u[i];
            }
            score = ((double)c[0] - lo) * ((double)c[0] - lo) + ((double)c[EO_NC - 1] - hi) * ((double)c[EO_NC - 1] - hi);
        }
        if (score < best_score) { best_score = score; best = k; }
    }
    float c[EO_NC];
    for (int j = 0; j < EO_NC; ++j) c[j] = eo_fp16_to_f32(M->pattern[best][j]);
    for (int i = 0; i < EO_G; ++i) sym[i] = (uint8_t)((i == p) ? 15 : eo_nearest(c, u[i]));
    *pstar_out = p; *qs_out = qs; *kp_out = best;
    if (err_out) *err_out = best_score;
    return EO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Block bit I/O.                                                                        */
/* reading (the block drawing is missing from the paper's text): stream bit k lives in    */
/* byte k>>3 at bit k&7; fixed-width fields are stored least-significant bit first;       */
/* codewords are stored first code bit (MSB of the canonical value) first.                */
/* ------------------------------------------------------------------------------------ */
static int eo_get_bit(const uint8_t* blk, int k) { return (k < EO_BITS) ? (blk[k >> 3] >> (k & 7)) & 1 : 0; }
static void eo_set_bit(uint8_t* blk, int k, int b) { if (b) blk[k >> 3] |= (uint8_t)(1u << (k & 7)); }

static void eo_put_field(uint8_t* blk, int pos, uint32_t v, int nbits)
{
    for (int i = 0; i < nbits; ++i) eo_set_bit(blk, pos + i, (v >> i) & 1);
}
static uint32_t eo_get_field(const uint8_t* blk, int pos, int nbits)
{
    uint32_t v = 0;
    for (int i = 0; i < nbits; ++i) v |= (uint32_t)eo_get_bit(blk, pos + i) << i;
    return v;
}
/* writes codeword bits that fall below bit 512; returns the new position (may exceed 512) */
static int eo_put_code(uint8_t* blk, int pos, uint32_t code, int len)
{
    for (int i = 0; i < len; ++i)
        if (pos + i < EO_BITS) eo_set_bit(blk, pos + i, (code >> (len - 1 - i)) & 1);
    return pos + len;
}
/* does the codeword (code, len) prefix the stream at pos?  bits at or past 512 read as 0 */
static int eo_code_matches(const uint8_t* blk, int pos, uint32_t code, int len)
{
    for (int i = 0; i < len; ++i)
        if (eo_get_bit(blk, pos + i) != (int)((code >> (len - 1 - i)) & 1)) return 0;
    return 1;
}

int eo_meta_check(const eo_meta* M)
{
    if (M->S < 2 || M->S > EO_MAXS || M->H != EO_H || M->e < -32 || M->e > 16) return EO_ERR_META;
    uint32_t kraft;
    uint16_t code[EO_MAXS];
    for (int k = 0; k < M->S; ++k) {
        if (M->kp_len[k] < 1 || M->kp_len[k] > EO_KP_MAXLEN) return EO_ERR_META;
        for (int j = 0; j < EO_NC; ++j) {
            float c = eo_fp16_to_f32(M->pattern[k][j]);
            if (!isfinite(c)) return EO_ERR_META;
            if (j && c < eo_fp16_to_f32(M->pattern[k][j - 1])) return EO_ERR_META;
        }
        for (int h = 0; h < EO_H; ++h) {
            for (int s = 0; s < EO_NSYM; ++s)
                if (M->cb_len[k][h][s] < 2 || M->cb_len[k][h][s] > 8) return EO_ERR_META;
            eo_canonical_codes(M->cb_len[k][h], EO_NSYM, 8, code, &kraft);
            if (kraft != 256) return EO_ERR_META;
        }
    }
    eo_canonical_codes(M->kp_len, M->S, EO_KP_MAXLEN, code, &kraft);
    if (kraft != (1u << EO_KP_MAXLEN)) return EO_ERR_META;
    return EO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Encoder (Fig. 4 steps 2, 5, 8, 9; Sec. 4.3).                                          */
/* Block layout, reading: [b0..b7] FP8 scale byte, [b8..b9] ID_HF, [b10..] ID_KP codeword, */
/* the 128 codewords in order, zero fill, pads in 15-bit slots growing down from b511:    */
/* pad j occupies [512-15(j+1), 512-15j), low 7 bits location, high 8 bits FP8 value.     */
/* ------------------------------------------------------------------------------------ */
typedef struct { int32_t pstar, kp, hf, n_fit, n_pad, end_bit; uint8_t qs; } eo_group_info;

int eo_encode_group(const eo_meta* M, const uint16_t* x16, int select, uint8_t* blk, uint8_t* sym_out,
                    eo_group_info* info)
{
    float u[EO_G];
    uint8_t sym[EO_G];
    int32_t p, kp; uint8_t qs;
    int rc = eo_quantize_group(M, x16, select, &p, &qs, u, &kp, sym, NULL);
    if (rc) return rc;

    /* step 8: the codebook with the shortest total length; ties to the lower id */
    int hf = 0, best_len = 1 << 30;
    for (int h = 0; h < EO_H; ++h) {
        int L = 0;
        for (int i = 0; i < EO_G; ++i) L += M->cb_len[kp][h][sym[i]];
        if (L < best_len) { best_len = L; hf = h; }
    }
    uint16_t kpcode[EO_MAXS], code[EO_NSYM];
    eo_canonical_codes(M->kp_len, M->S, EO_KP_MAXLEN, kpcode, NULL);
    eo_canonical_codes(M->cb_len[kp][hf], EO_NSYM, 8, code, NULL);

    memset(blk, 0, EO_BLOCK);
    eo_put_field(blk, 0, qs, 8);
    eo_put_field(blk, 8, (uint32_t)hf, 2);
    int pos = eo_put_code(blk, 10, kpcode[kp], M->kp_len[kp]);
    /* step 9, clip: reading: literal truncation of the bit string at bit 512 */
    int n_fit = 0, end = pos;
    for (int i = 0; i < EO_G; ++i) {
        pos = eo_put_code(blk, pos, code[sym[i]], M->cb_len[kp][hf][sym[i]]);
        if (pos <= EO_BITS) { n_fit = i + 1; end = pos; } else break;
    }
    int n_pad = 0;
    if (n_fit == EO_G) {
        /* step 9, pad: the other elements from the second largest |x| downwards, as many
           15-bit slots as fit, at most 16 */
        n_pad = (EO_BITS - end) / EO_PAD_BITS;
        if (n_pad > EO_MAX_PADS) n_pad = EO_MAX_PADS;
        float T = (float)ldexp(1.0, M->e);
        uint8_t taken[EO_G] = {0};
        taken[p] = 1;
        for (int j = 0; j < n_pad; ++j) {
            int loc = -1; float mag = -1.0f;
            for (int i = 0; i < EO_G; ++i) {
                float a = fabsf(eo_fp16_to_f32(x16[i]));
                if (!taken[i] && a > mag) { mag = a; loc = i; }
            }
            taken[loc] = 1;
            uint8_t val = eo_e4m3_from_f32(eo_fp16_to_f32(x16[loc]) / T);
            eo_put_field(blk, EO_BITS - EO_PAD_BITS * (j + 1), (uint32_t)loc | ((uint32_t)val << 7), EO_PAD_BITS);
        }
    }
    if (sym_out) memcpy(sym_out, sym, EO_G);
    if (info) { info->pstar = p; info->kp = kp; info->hf = hf; info->n_fit = n_fit; info->n_pad = n_pad;
                info->end_bit = end; info->qs = qs; }
    return EO_OK;
}

int eo_encode(const eo_meta* M, const uint16_t* x16, uint64_t n_groups, int select, uint8_t* blocks, eo_stats* st)
{
    int rc = eo_meta_check(M);
    if (rc) return rc;
    if (st) memset(st, 0, sizeof *st);
    for (uint64_t g = 0; g < n_groups; ++g) {
        eo_group_info info; uint8_t sym[EO_G];
        rc = eo_encode_group(M, x16 + g * EO_G, select, blocks + g * EO_BLOCK, sym, &info);
        if (rc) return rc;
        if (st) {
            st->n_groups++;
            if (info.n_fit < EO_G) { st->clipped_groups++; st->clipped_values += (uint64_t)(EO_G - info.n_fit); }
            if (info.n_pad) { st->padded_groups++; st->padded_values += (uint64_t)info.n_pad; }
            st->total_bits += (uint64_t)info.end_bit;
            st->kp_usage[info.kp]++; st->hf_usage[info.hf]++;
            for (int i = 0; i < EO_G; ++i) st->sym_count[sym[i]]++;
        }
    }
    return EO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Decoder (Sec. 4.2): total function of the 64 bytes and the metadata.                  */
/* ------------------------------------------------------------------------------------ */
int eo_decode_block(const eo_meta* M, const uint8_t* blk, uint16_t* out16, uint8_t* sym_out, eo_group_info* info)
{
    float T = (float)ldexp(1.0, M->e);
    /* pattern retriever: scale byte, ID_HF, Huffman-coded ID_KP */
    uint8_t qs = (uint8_t)eo_get_field(blk, 0, 8);
    int hf = (int)eo_get_field(blk, 8, 2);
    uint16_t kpcode[EO_MAXS], code[EO_NSYM];
    eo_canonical_codes(M->kp_len, M->S, EO_KP_MAXLEN, kpcode, NULL);
    int kp = -1;
    for (int k = 0; k < M->S; ++k)
        if (eo_code_matches(blk, 10, kpcode[k], M->kp_len[k])) { kp = k; break; }
    if (kp < 0) return EO_ERR_META;   /* cannot happen with a complete code */
    int pos = 10 + M->kp_len[kp];
    float s = fabsf(eo_e4m3_to_f32(qs)) * T;    /* FP8 -> FP16 by exponent adjust */
    eo_canonical_codes(M->cb_len[kp][hf], EO_NSYM, 8, code, NULL);

    /* Huffman decode: until 128 symbols, or until the next codeword would cross bit 512 */
    uint8_t sym[EO_G];
    int n = 0;
    while (n < EO_G) {
        int found = -1;
        for (int c = 0; c < EO_NSYM; ++c)
            if (eo_code_matches(blk, pos, code[c], M->cb_len[kp][hf][c])) { found = c; break; }
        if (found < 0) return EO_ERR_META;  /* cannot happen with a complete code */
        int L = M->cb_len[kp][hf][found];
        if (pos + L > EO_BITS) break;
        sym[n++] = (uint8_t)found;
        pos += L;
    }
    /* mapper: centroid x scale with one fp32 product and one rounding; index 15 restores the
       signed abs-max; clipped positions read +0 */
    for (int i = 0; i < EO_G; ++i) {
        if (i >= n) out16[i] = 0;
        else if (sym[i] == 15) out16[i] = eo_f32_to_fp16(eo_e4m3_to_f32(qs) * T);
        else out16[i] = eo_f32_to_fp16(eo_fp16_to_f32(M->pattern[kp][sym[i]]) * s);
    }
    /* outliers: only a complete group carries pads; a later pad overrides an earlier one */
    int n_pad = 0;
    if (n == EO_G) {
        n_pad = (EO_BITS - pos) / EO_PAD_BITS;
        if (n_pad > EO_MAX_PADS) n_pad = EO_MAX_PADS;
        for (int j = 0; j < n_pad; ++j) {
            uint32_t f = eo_get_field(blk, EO_BITS - EO_PAD_BITS * (j + 1), EO_PAD_BITS);
            out16[f & 127] = eo_f32_to_fp16(eo_e4m3_to_f32((uint8_t)(f >> 7)) * T);
        }
    }
    if (sym_out) { memcpy(sym_out, sym, (size_t)n); memset(sym_out + n, 0xff, (size_t)(EO_G - n)); }
    if (info) { info->pstar = -1; info->kp = kp; info->hf = hf; info->n_fit = n; info->n_pad = n_pad;
                info->end_bit = pos; info->qs = qs; }
    return EO_OK;
}

int eo_decode(const eo_meta* M, const uint8_t* blocks, uint64_t n_groups, uint16_t* out16)
{
    int rc = eo_meta_check(M);
    if (rc) return rc;
    for (uint64_t g = 0; g < n_groups; ++g) {
        rc = eo_decode_block(M, blocks + g * EO_BLOCK, out16 + g * EO_G, NULL, NULL);
        if (rc) return rc;
    }
    return EO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Consumers (Sec. 2.1): fp64 dot products over the decompressed fp16 values.            */
/* ------------------------------------------------------------------------------------ */

/* y[b][n] = sum_k W~[n][k] x[b][k]; W row-major [n_out][k], groups along k.
   Also writes sum_k |W~ x| per output into yabs (may be NULL) for the error metric. */
int eo_gemv(const eo_meta* M, const uint8_t* blocks, int n_out, int k, const uint16_t* x16, int batch,
            double* y, double* yabs)
{
    if (k % EO_G) return EO_ERR_ARG;
    int rc = eo_meta_check(M);
    if (rc) return rc;
    int kb = k / EO_G;
    uint16_t w16[EO_G];
    for (int b = 0; b < batch; ++b)
        for (int n = 0; n < n_out; ++n) { y[(size_t)b * n_out + n] = 0.0; if (yabs) yabs[(size_t)b * n_out + n] = 0.0; }
    for (int n = 0; n < n_out; ++n)
        for (int j = 0; j < kb; ++j) {
            rc = eo_decode_block(M, blocks + ((size_t)n * kb + j) * EO_BLOCK, w16, NULL, NULL);
            if (rc) return rc;
            for (int b = 0; b < batch; ++b) {
                double acc = 0.0, aacc = 0.0;
                for (int i = 0; i < EO_G; ++i) {
                    double t = (double)eo_fp16_to_f32(w16[i]) * (double)eo_fp16_to_f32(x16[(size_t)b * k + j * EO_G + i]);
                    acc += t; aacc += fabs(t);
                }
                y[(size_t)b * n_out + n] += acc;
                if (yabs) yabs[(size_t)b * n_out + n] += aacc;
            }
        }
    return EO_OK;
}

/* scores[b][hq][t] = scale * sum_d q[b][hq][d] * K~[b][hq / q_per_kv][t][d]   (Eq. 3: QK^T / sqrt(d_k));
   one group = the 128-wide head vector of one token; blocks ordered [batch][kv_head][seq]. */
int eo_attn_scores(const eo_meta* M, const uint8_t* kblocks, int batch, int n_kv_heads, int seq, int q_per_kv,
                   const uint16_t* q16, double scale, double* scores, double* sabs)
{
    int rc = eo_meta_check(M);
    if (rc) return rc;
    uint16_t k16[EO_G];
    int n_q = n_kv_heads * q_per_kv;
    for (int b = 0; b < batch; ++b)
        for (int h = 0; h < n_kv_heads; ++h)
            for (int t = 0; t < seq; ++t) {
                size_t g = ((size_t)b * n_kv_heads + h) * (size_t)seq + t;
                rc = eo_decode_block(M, kblocks + g * EO_BLOCK, k16, NULL, NULL);
                if (rc) return rc;
                for (int r = 0; r < q_per_kv; ++r) {
                    int hq = h * q_per_kv + r;
                    const uint16_t* q = q16 + ((size_t)b * n_q + hq) * EO_G;
                    double acc = 0.0, aacc = 0.0;
                    for (int d = 0; d < EO_G; ++d) {
                        double tt = (double)eo_fp16_to_f32(q[d]) * (double)eo_fp16_to_f32(k16[d]);
                        acc += tt; aacc += fabs(tt);
                    }
                    scores[((size_t)b * n_q + hq) * (size_t)seq + t] = scale * acc;
                    if (sabs) sabs[((size_t)b * n_q + hq) * (size_t)seq + t] = fabs(scale) * aacc;
                }
            }
    return EO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Calibration (Fig. 4 steps 2-7 on a calibration tensor).                               */
/* ------------------------------------------------------------------------------------ */
static int eo_cmp_double(const void* a, const void* b)
{
    double x = *(const double*)a, y = *(const double*)b;
    return (x > y) - (x < y);
}
typedef struct { double v, w; } eo_vw;
static int eo_cmp_vw(const void* a, const void* b)
{
    double x = ((const eo_vw*)a)->v, y = ((const eo_vw*)b)->v;
    return (x > y) - (x < y);
}

/* Step 3 for one group: normalise by the FP8-rounded abs-max, drop the abs-max, exact
   15-means on the 127 others.  pattern15 receives the ascending centroids. */
int eo_group_pattern(const uint16_t* x16, int e, const float* weights_or_null, double* pattern15)
{
    float T = (float)ldexp(1.0, e);
    float x[EO_G];
    int p = 0;
    for (int i = 0; i < EO_G; ++i) {
        x[i] = eo_fp16_to_f32(x16[i]);
        if (!isfinite(x[i])) return EO_ERR_NONFINITE;
        if (fabsf(x[i]) > fabsf(x[p])) p = i;
    }
    float s = fabsf(eo_e4m3_to_f32(eo_e4m3_from_f32(x[p] / T))) * T;
    eo_vw vw[EO_G - 1];
    int m = 0;
    for (int i = 0; i < EO_G; ++i) {
        if (i == p) continue;
        vw[m].v = (s == 0.0f) ? 0.0 : (double)(x[i] / s);
        vw[m].w = weights_or_null ? (double)weights_or_null[i] : 1.0;
        ++m;
    }
    qsort(vw, EO_G - 1, sizeof(eo_vw), eo_cmp_vw);
    double v[EO_G - 1], w[EO_G - 1];
    for (int i = 0; i < EO_G - 1; ++i) { v[i] = vw[i].v; w[i] = vw[i].w; }
    (void)eo_cmp_double;
    eo_kmeans1d(v, weights_or_null ? w : NULL, EO_G - 1, EO_NC, pattern15);
    return EO_OK;
}

/* Full calibration.  weights: NULL or one non-negative weight per element of a group
   (128 floats, the same for every group).  The per-tensor exponent is taken from the
   calibration tensor; eo_set_exponent() replaces it for the tensor actually encoded. */
int eo_calibrate(const uint16_t* calib16, uint64_t n_groups, const float* weights, int S, int H, uint64_t seed,
                 int select, int lloyd_iters, eo_meta* M)
{
    if (S < 2 || S > EO_MAXS || H != EO_H || n_groups < (uint64_t)S) return EO_ERR_ARG;
    memset(M, 0, sizeof *M);
    M->S = S; M->H = H;
    int rc = eo_choose_exponent(calib16, n_groups * EO_G, &M->e);
    if (rc) return rc;
    int n = (int)n_groups;

    /* steps 2-3: per-group patterns */
    double* pats = (double*)malloc(sizeof(double) * (size_t)n * EO_NC);
    for (int g = 0; g < n; ++g) {
        rc = eo_group_pattern(calib16 + (size_t)g * EO_G, M->e, weights, pats + (size_t)g * EO_NC);
        if (rc) { free(pats); return rc; }
    }
    /* step 4: S shared patterns; cluster means of ascending vectors are ascending */
    double* centre = (double*)malloc(sizeof(double) * (size_t)S * EO_NC);
    int32_t* assign = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    eo_lloyd(pats, n, EO_NC, S, seed, lloyd_iters, centre, assign, NULL);
    for (int k = 0; k < S; ++k)
        for (int j = 0; j < EO_NC; ++j) M->pattern[k][j] = eo_f32_to_fp16((float)centre[(size_t)k * EO_NC + j]);
    free(centre); free(pats);

    /* provisional codes so that the metadata is complete while step 5 runs */
    for (int k = 0; k < S; ++k) {
        M->kp_len[k] = 0;
        for (int h = 0; h < H; ++h) for (int s = 0; s < EO_NSYM; ++s) M->cb_len[k][h][s] = 4;
    }
    /* step 5 on the calibration groups: pattern choice and symbols */
    int32_t* kp = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    double* hist = (double*)calloc((size_t)n * EO_NSYM, sizeof(double));
    for (int g = 0; g < n; ++g) {
        float u[EO_G]; uint8_t sym[EO_G]; int32_t p; uint8_t qs;
        rc = eo_quantize_group(M, calib16 + (size_t)g * EO_G, select, &p, &qs, u, &kp[g], sym, NULL);
        if (rc) { free(kp); free(hist); free(assign); return rc; }
        for (int i = 0; i < EO_G; ++i) hist[(size_t)g * EO_NSYM + sym[i]] += 1.0 / EO_G;
    }
    /* steps 6-7 per pattern: H representative histograms -> H codebooks */
    double usage[EO_MAXS];
    double* sub = (double*)malloc(sizeof(double) * (size_t)n * EO_NSYM);
    int32_t* sub_assign = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    for (int k = 0; k < S; ++k) {
        int m = 0;
        for (int g = 0; g < n; ++g)
            if (kp[g] == k) { memcpy(sub + (size_t)m * EO_NSYM, hist + (size_t)g * EO_NSYM, sizeof(double) * EO_NSYM); ++m; }
        usage[k] = (double)m + 1.0;
        double rep[EO_H][EO_NSYM];
        if (m >= H) {
            double cen[EO_H * EO_NSYM];
            eo_lloyd(sub, m, EO_NSYM, H, seed + 1 + (uint64_t)k, lloyd_iters, cen, sub_assign, NULL);
            memcpy(rep, cen, sizeof rep);
        } else {
            /* reading: fewer than H member groups -> every codebook uses the mean histogram
               (uniform when the pattern is unused) */
            double mean[EO_NSYM];
            for (int s = 0; s < EO_NSYM; ++s) {
                mean[s] = 0.0;
                for (int g = 0; g < m; ++g) mean[s] += sub[(size_t)g * EO_NSYM + s];
                mean[s] = m ? mean[s] / m : 1.0 / EO_NSYM;
            }
            for (int h = 0; h < H; ++h) memcpy(rep[h], mean, sizeof mean);
        }
        for (int h = 0; h < H; ++h) {
            rc = eo_huffman_2_8(rep[h], M->cb_len[k][h]);
            if (rc) { free(kp); free(hist); free(assign); free(sub); free(sub_assign); return rc; }
        }
    }
    /* ID_KP code from pattern usage + 1 */
    rc = eo_huffman_limited(usage, S, EO_KP_MAXLEN, M->kp_len);
    free(kp); free(hist); free(assign); free(sub); free(sub_assign);
    if (rc) return rc;
    return eo_meta_check(M);
}

int eo_set_exponent(eo_meta* M, const uint16_t* x16, uint64_t n_values) { return eo_choose_exponent(x16, n_values, &M->e); }

int eo_sizeof_meta(void) { return (int)sizeof(eo_meta); }
int eo_sizeof_stats(void) { return (int)sizeof(eo_stats); }
int eo_sizeof_info(void) { return (int)sizeof(eo_group_info); }

/* ------------------------------------------------------------------------------------ */
/* 2x activation format (Sec. 3.2 "Activation Compression", Sec. 4.2/4.3 low-ratio units): */
/* 64 values -> 64 bytes; every byte holds a 7-bit quantised value, the eighth bit of the   */
/* bytes carries a 16-bit scale factor and a 16-bit zero point, one bit per byte.           */
/* reading (the paper gives the field widths only): byte i = q_i in its low 7 bits          */
/* (two's complement, -64..63: the decompressor sign-extends 7 -> 8 bits) and metadata bit  */
/* i in bit 7; metadata bits 0..15 = fp16 scale (lsb first), 16..31 = fp16 zero point,       */
/* 32..63 = 0.  scale = fp16((max - min) / 127), zero = fp16(min + 64 * scale) (so q = -64   */
/* is the group minimum), q = clamp(rint((x - zero) * (1 / scale)), -64, 63) in fp32 with    */
/* the rounded scale and zero -- a multiply by the reciprocal, as in the compressor's        */
/* "multiply-and-round circuit" (Sec. 4.3, low-ratio compressor); 1 / scale is one fp32      */
/* division per group; a zero scale stores q = 0.  Dequantisation is one fp32 fused          */
/* multiply-add rounded to fp16 (the "two operations" of the decompressor): q * scale + zero. */
/* Parity unpinned: these choices are this build's definition.  Inputs must be finite.      */
/* ------------------------------------------------------------------------------------ */
#define EO_ACT_G 64

int eo_act_encode_group(const uint16_t* x16, uint8_t* blk)
{
    float x[EO_ACT_G], lo = INFINITY, hi = -INFINITY;
    for (int i = 0; i < EO_ACT_G; ++i) {
        x[i] = eo_fp16_to_f32(x16[i]);
        if (!isfinite(x[i])) return EO_ERR_NONFINITE;
        if (x[i] < lo) lo = x[i];
        if (x[i] > hi) hi = x[i];
    }
    uint16_t scale16 = eo_f32_to_fp16((hi - lo) / 127.0f);
    float scale = eo_fp16_to_f32(scale16);
    uint16_t zero16 = eo_f32_to_fp16(lo + 64.0f * scale);
    float zero = eo_fp16_to_f32(zero16);
    uint32_t meta_lo = (uint32_t)scale16 | ((uint32_t)zero16 << 16);
    for (int i = 0; i < EO_ACT_G; ++i) {
        int q = 0;
        if (scale > 0.0f && isfinite(scale)) {
            float inv = 1.0f / scale;
            float r = rintf((x[i] - zero) * inv);
            q = r < -64.0f ? -64 : r > 63.0f ? 63 : (int)r;
        }
        int mbit = (i < 32) ? (int)((meta_lo >> i) & 1u) : 0;
        blk[i] = (uint8_t)(((unsigned)q & 0x7fu) | ((unsigned)mbit << 7));
    }
    return EO_OK;
}

void eo_act_decode_group(const uint8_t* blk, uint16_t* out16)
{
    uint32_t meta_lo = 0;
    for (int i = 0; i < 32; ++i) meta_lo |= (uint32_t)(blk[i] >> 7) << i;
    float scale = eo_fp16_to_f32((uint16_t)(meta_lo & 0xffffu));
    float zero = eo_fp16_to_f32((uint16_t)(meta_lo >> 16));
    for (int i = 0; i < EO_ACT_G; ++i) {
        int q = blk[i] & 0x7f;
        if (q & 0x40) q -= 128;                 /* sign extension of the 7-bit value */
        out16[i] = eo_f32_to_fp16(fmaf((float)q, scale, zero));
    }
}

int eo_act_encode(const uint16_t* x16, uint64_t n_groups, uint8_t* blocks)
{
    for (uint64_t g = 0; g < n_groups; ++g) {
        int rc = eo_act_encode_group(x16 + g * EO_ACT_G, blocks + g * 64);
        if (rc) return rc;
    }
    return EO_OK;
}

void eo_act_decode(const uint8_t* blocks, uint64_t n_groups, uint16_t* out16)
{
    for (uint64_t g = 0; g < n_groups; ++g) eo_act_decode_group(blocks + g * 64, out16 + g * EO_ACT_G);
}

/* ------------------------------------------------------------------------------------ */
/* Attention output over a compressed V cache (Eq. 3: softmax(QK^T / sqrt(d_k)) V):       */
/* out[b][hq][d] = sum_t softmax_t(scores[b][hq][:])[t] * V~[b][hq / q_per_kv][t][d], in   */
/* fp64 over the decompressed fp16 values.  scores are the fp32 logits (already scaled).   */
/* outabs receives sum_t p_t |V~| for the error metric.                                    */
/* ------------------------------------------------------------------------------------ */
int eo_attn_values(const eo_meta* M, const uint8_t* vblocks, int batch, int n_kv_heads, int seq, int q_per_kv,
                   const float* scores, double* out, double* outabs)
{
    int rc = eo_meta_check(M);
    if (rc) return rc;
    int n_q = n_kv_heads * q_per_kv;
    uint16_t v16[EO_G];
    double* p = (double*)malloc(sizeof(double) * (size_t)seq * (size_t)q_per_kv);
    for (int b = 0; b < batch; ++b)
        for (int h = 0; h < n_kv_heads; ++h) {
            for (int r = 0; r < q_per_kv; ++r) {
                const float* s = scores + ((size_t)b * n_q + h * q_per_kv + r) * (size_t)seq;
                double mx = -INFINITY, sum = 0.0;
                for (int t = 0; t < seq; ++t) if (s[t] > mx) mx = s[t];
                for (int t = 0; t < seq; ++t) { p[(size_t)r * seq + t] = exp((double)s[t] - mx); sum += p[(size_t)r * seq + t]; }
                for (int t = 0; t < seq; ++t) p[(size_t)r * seq + t] /= sum;
                double* o = out + ((size_t)b * n_q + h * q_per_kv + r) * EO_G;
                double* oa = outabs ? outabs + ((size_t)b * n_q + h * q_per_kv + r) * EO_G : NULL;
                for (int d = 0; d < EO_G; ++d) { o[d] = 0.0; if (oa) oa[d] = 0.0; }
            }
            for (int t = 0; t < seq; ++t) {
                size_t g = ((size_t)b * n_kv_heads + h) * (size_t)seq + t;
                rc = eo_decode_block(M, vblocks + g * EO_BLOCK, v16, NULL, NULL);
                if (rc) { free(p); return rc; }
                for (int r = 0; r < q_per_kv; ++r) {
                    double* o = out + ((size_t)b * n_q + h * q_per_kv + r) * EO_G;
                    double* oa = outabs ? outabs + ((size_t)b * n_q + h * q_per_kv + r) * EO_G : NULL;
                    double pt = p[(size_t)r * seq + t];
                    for (int d = 0; d < EO_G; ++d) {
                        double v = (double)eo_fp16_to_f32(v16[d]);
                        o[d] += pt * v;
                        if (oa) oa[d] += pt * fabs(v);
                    }
                }
            }
        }
    free(p);
    return EO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Variable-length container (the alternative layout without clipping and padding): the    */
/* same per-group fields -- scale byte, ID_HF, ID_KP codeword, 128 codewords (Sec. 3.2) -- */
/* written back to back into one bit stream, plus an index of where every group starts.    */
/* reading (the paper only has the fixed 64-byte block; this layout is this build's):      */
/* stream bit k = bit k&7 of byte k>>3 as in the block; the groups of one chunk of 4096    */
/* groups follow each other without gaps; offsets[g] is the absolute start bit of group g  */
/* and offsets[n_groups] the total length.  Nothing is clipped and nothing is padded.      */
/* The decoder of group g sees the stream bits in [offsets[g], offsets[g+1]) and zeros      */
/* after them, so any stream and any offsets decode to something.                           */
/* ------------------------------------------------------------------------------------ */
#define EO_VAR_MAX_BITS (10 + EO_KP_MAXLEN + EO_G * 8)

static int eo_sget_bit(const uint8_t* s, uint64_t k) { return (s[k >> 3] >> (k & 7)) & 1; }
static void eo_sset_bit(uint8_t* s, uint64_t k, int b) { if (b) s[k >> 3] |= (uint8_t)(1u << (k & 7)); }

/* stream must be zero-initialised and hold (total bits + 7) / 8 bytes; returns the bit count through offsets */
int eo_var_encode(const eo_meta* M, const uint16_t* x16, uint64_t n_groups, int select, uint8_t* stream, uint64_t* offsets)
{
    int rc = eo_meta_check(M);
    if (rc) return rc;
    uint16_t kpcode[EO_MAXS], code[EO_NSYM];
    eo_canonical_codes(M->kp_len, M->S, EO_KP_MAXLEN, kpcode, NULL);
    uint64_t pos = 0;
    for (uint64_t g = 0; g < n_groups; ++g) {
        float u[EO_G]; uint8_t sym[EO_G]; int32_t p, kp; uint8_t qs;
        rc = eo_quantize_group(M, x16 + g * EO_G, select, &p, &qs, u, &kp, sym, NULL);
        if (rc) return rc;
        int hf = 0, best_len = 1 << 30;
        for (int h = 0; h < EO_H; ++h) {
            int L = 0;
            for (int i = 0; i < EO_G; ++i) L += M->cb_len[kp][h][sym[i]];
            if (L < best_len) { best_len = L; hf = h; }
        }
        eo_canonical_codes(M->cb_len[kp][hf], EO_NSYM, 8, code, NULL);
        offsets[g] = pos;
        for (int i = 0; i < 8; ++i) eo_sset_bit(stream, pos++, (qs >> i) & 1);
        for (int i = 0; i < 2; ++i) eo_sset_bit(stream, pos++, (hf >> i) & 1);
        for (int i = 0; i < M->kp_len[kp]; ++i) eo_sset_bit(stream, pos++, (kpcode[kp] >> (M->kp_len[kp] - 1 - i)) & 1);
        for (int n = 0; n < EO_G; ++n) {
            int L = M->cb_len[kp][hf][sym[n]];
            for (int i = 0; i < L; ++i) eo_sset_bit(stream, pos++, (code[sym[n]] >> (L - 1 - i)) & 1);
        }
    }
    offsets[n_groups] = pos;
    return EO_OK;
}

/* group g reads bits below offsets[g+1] (and below the total length); everything else reads as 0 */
int eo_var_decode(const eo_meta* M, const uint8_t* stream, const uint64_t* offsets, uint64_t n_groups, uint16_t* out16)
{
    int rc = eo_meta_check(M);
    if (rc) return rc;
    float T = (float)ldexp(1.0, M->e);
    uint16_t kpcode[EO_MAXS], code[EO_NSYM];
    eo_canonical_codes(M->kp_len, M->S, EO_KP_MAXLEN, kpcode, NULL);
    uint64_t total = offsets[n_groups];
#define EO_SBIT(k) ((k) < limit ? eo_sget_bit(stream, (k)) : 0)
    for (uint64_t g = 0; g < n_groups; ++g) {
        uint64_t pos = offsets[g];
        uint64_t limit = offsets[g + 1] < total ? offsets[g + 1] : total;
        uint32_t qs = 0, hf = 0;
        for (int i = 0; i < 8; ++i) qs |= (uint32_t)EO_SBIT(pos + i) << i;
        for (int i = 0; i < 2; ++i) hf |= (uint32_t)EO_SBIT(pos + 8 + i) << i;
        pos += 10;
        int kp = -1;
        for (int k = 0; k < M->S && kp < 0; ++k) {
            int ok = 1;
            for (int i = 0; i < M->kp_len[k] && ok; ++i) ok = EO_SBIT(pos + i) == (int)((kpcode[k] >> (M->kp_len[k] - 1 - i)) & 1);
            if (ok) kp = k;
        }
        if (kp < 0) return EO_ERR_META;
        pos += M->kp_len[kp];
        float s = fabsf(eo_e4m3_to_f32((uint8_t)qs)) * T;
        eo_canonical_codes(M->cb_len[kp][hf], EO_NSYM, 8, code, NULL);
        for (int n = 0; n < EO_G; ++n) {
            int found = -1;
            for (int c = 0; c < EO_NSYM && found < 0; ++c) {
                int L = M->cb_len[kp][hf][c], ok = 1;
                for (int i = 0; i < L && ok; ++i) ok = EO_SBIT(pos + i) == (int)((code[c] >> (L - 1 - i)) & 1);
                if (ok) found = c;
            }
            if (found < 0) return EO_ERR_META;
            pos += M->cb_len[kp][hf][found];
            out16[g * EO_G + n] = found == 15 ? eo_f32_to_fp16(eo_e4m3_to_f32((uint8_t)qs) * T)
                                             : eo_f32_to_fp16(eo_fp16_to_f32(M->pattern[kp][found]) * s);
        }
    }
#undef EO_SBIT
    return EO_OK;
}
