// ecco_host.cpp -- host side of the library: metadata, calibration (Fig. 4 steps 1-7), the
// threaded block encoder (Fig. 4 steps 2, 5, 8, 9; Sec. 4.3) and the device metadata image with
// the prebuilt decode tables (Sec. 4.2, "loaded once").  No CUDA in this file.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <memory>
#include <mutex>
#include <new>
#include <numeric>
#include <thread>
#include <vector>

#include <sched.h>

#include "../../include/ecco.h"
#include "ecco_format.h"

using namespace ecco;

// ---------------------------------------------------------------------------------------------
// number formats
// ---------------------------------------------------------------------------------------------
namespace {

float g_half_table[65536];
float g_fp8_table[256];
std::once_flag g_tables_once;

void build_tables()
{
    for (uint32_t h = 0; h < 65536; ++h) {
        uint32_t sign = (h & 0x8000u) << 16, ex = (h >> 10) & 31u, man = h & 1023u, bits;
        if (ex == 0) {
            float v = std::ldexp(static_cast<float>(man), -24);
            std::memcpy(&bits, &v, 4);
            bits |= sign;
        } else if (ex == 31) {
            bits = sign | 0x7f800000u | (man << 13);
        } else {
            bits = sign | ((ex + 112u) << 23) | (man << 13);
        }
        std::memcpy(&g_half_table[h], &bits, 4);
    }
    for (uint32_t b = 0; b < 256; ++b) {
        uint32_t ex = (b >> 3) & 15u, man = b & 7u;
        float v = ex ? std::ldexp(static_cast<float>(8 + man), static_cast<int>(ex) - 10)
                     : std::ldexp(static_cast<float>(man), -9);
        g_fp8_table[b] = (b & 0x80u) ? -v : v;
    }
}
inline void ensure_tables() { std::call_once(g_tables_once, build_tables); }
inline float half_to_float(uint16_t h) { return g_half_table[h]; }
inline float fp8_to_float(uint8_t b) { return g_fp8_table[b]; }

// float -> OCP E4M3, round to nearest even, saturating at +-448 (0x7E); works on the raw bits
inline uint8_t float_to_fp8(float f)
{
    uint32_t x;
    std::memcpy(&x, &f, 4);
    const uint8_t sign = static_cast<uint8_t>((x >> 24) & 0x80u);
    const uint32_t ax = x & 0x7fffffffu;
    if (ax >= 0x43e00000u) return sign | 0x7e;               // >= 448, inf, nan
    if (ax < 0x3c800000u) {                                  // below 2^-6: subnormal grid of 2^-9
        float a;
        std::memcpy(&a, &ax, 4);
        return sign | static_cast<uint8_t>(std::nearbyintf(a * 512.0f));
    }
    uint32_t r = ax + 0x7ffffu + ((ax >> 20) & 1u);          // ties to even at mantissa bit 20
    r = (r >> 20) - ((127u - 7u) << 3);
    return sign | static_cast<uint8_t>(r > 0x7eu ? 0x7eu : r);
}

inline uint32_t bit_reverse(uint32_t v, int n)
{
    uint32_t r = 0;
    for (int i = 0; i < n; ++i) r |= ((v >> i) & 1u) << (n - 1 - i);
    return r;
}

// canonical code: symbols by (length, id), consecutive values; returns false unless Kraft == 1
bool canonical(const uint8_t* len, int n, int maxlen, uint16_t* code)
{
    uint32_t next = 0, kraft = 0;
    int prev = 0;
    for (int L = 1; L <= maxlen; ++L)
        for (int s = 0; s < n; ++s)
            if (len[s] == L) {
                if (prev) next = (next + 1) << (L - prev);
                code[s] = static_cast<uint16_t>(next);
                prev = L;
                kraft += 1u << (maxlen - L);
            }
    return kraft == (1u << maxlen);
}

int available_cores()
{
    cpu_set_t set;
    CPU_ZERO(&set);
    if (sched_getaffinity(0, sizeof(set), &set) == 0) {
        int n = CPU_COUNT(&set);
        if (n > 0) return n;
    }
    unsigned hc = std::thread::hardware_concurrency();
    return hc ? static_cast<int>(hc) : 1;
}

template <class F>
void parallel_ranges(uint64_t n, int threads, F&& fn)
{
    if (threads <= 0) threads = available_cores();
    threads = static_cast<int>(std::min<uint64_t>(static_cast<uint64_t>(threads), std::max<uint64_t>(1, n / 64)));
    if (threads <= 1) { fn(0, uint64_t{0}, n); return; }
    std::vector<std::thread> pool;
    for (int t = 0; t < threads; ++t)
        pool.emplace_back([&, t] { fn(t, n * t / threads, n * (t + 1) / threads); });
    for (auto& th : pool) th.join();
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// metadata
// ---------------------------------------------------------------------------------------------
struct ecco_meta {
    int32_t S = 0, e = 0;
    uint16_t pattern[kMaxPatterns][16] = {};
    uint8_t cb_len[kMaxPatterns][kCodebooks][kSymbols] = {};
    uint8_t kp_len[kMaxPatterns] = {};
    // derived
    float pattern_f[kMaxPatterns][kCentroids] = {};
    uint16_t cb_rev[kMaxPatterns][kCodebooks][kSymbols] = {};   // bit-reversed codewords (stream order, lsb first)
    uint16_t kp_rev[kMaxPatterns] = {};
};

namespace {

int derive(ecco_meta* m)
{
    ensure_tables();
    if (m->S < 2 || m->S > kMaxPatterns || m->e < kExpMin || m->e > kExpMax) return ECCO_ERR_BAD_META;
    uint16_t code[kMaxPatterns];
    for (int k = 0; k < m->S; ++k) {
        if (m->kp_len[k] < 1 || m->kp_len[k] > kKpMaxLen) return ECCO_ERR_BAD_META;
        for (int j = 0; j < kCentroids; ++j) {
            float c = half_to_float(m->pattern[k][j]);
            if (!std::isfinite(c)) return ECCO_ERR_BAD_META;
            if (j && c < m->pattern_f[k][j - 1]) return ECCO_ERR_BAD_META;
            m->pattern_f[k][j] = c;
        }
        m->pattern[k][15] = 0;
        for (int h = 0; h < kCodebooks; ++h) {
            for (int s = 0; s < kSymbols; ++s)
                if (m->cb_len[k][h][s] < kMinLen || m->cb_len[k][h][s] > kMaxLen) return ECCO_ERR_BAD_META;
            if (!canonical(m->cb_len[k][h], kSymbols, kMaxLen, code)) return ECCO_ERR_BAD_META;
            for (int s = 0; s < kSymbols; ++s)
                m->cb_rev[k][h][s] = static_cast<uint16_t>(bit_reverse(code[s], m->cb_len[k][h][s]));
        }
    }
    if (!canonical(m->kp_len, m->S, kKpMaxLen, code)) return ECCO_ERR_BAD_META;
    for (int k = 0; k < m->S; ++k) m->kp_rev[k] = static_cast<uint16_t>(bit_reverse(code[k], m->kp_len[k]));
    return ECCO_OK;
}

// smallest e in [kExpMin, kExpMax] with max|x| <= 448 * 2^e; non-finite input is an error
int fit_exponent(const uint16_t* x, uint64_t n, int threads, int32_t* e_out)
{
    ensure_tables();
    std::atomic<bool> bad{false};
    std::vector<uint16_t> part(static_cast<size_t>(std::max(1, threads > 0 ? threads : available_cores())), 0);
    parallel_ranges(n, static_cast<int>(part.size()), [&](int t, uint64_t lo, uint64_t hi) {
        uint16_t mx = 0;                                   // |x| orders like its 15-bit pattern
        for (uint64_t i = lo; i < hi; ++i) {
            uint16_t a = x[i] & 0x7fffu;
            if (a >= 0x7c00u) { bad = true; return; }
            if (a > mx) mx = a;
        }
        part[static_cast<size_t>(t)] = mx;
    });
    if (bad) return ECCO_ERR_NONFINITE_INPUT;
    double mx = half_to_float(*std::max_element(part.begin(), part.end()));
    int e = kExpMin;
    while (e < kExpMax && mx > 448.0 * std::ldexp(1.0, e)) ++e;
    *e_out = e;
    return ECCO_OK;
}

// ---------------------------------------------------------------------------------------------
// per-group quantisation (Fig. 4 steps 2 and 5)
// ---------------------------------------------------------------------------------------------
struct Quantized {
    int pstar, kp;
    uint8_t qs;
    uint8_t sym[kGroup];
};

struct Scratch {
    float x[kGroup], u[kGroup];
    int order[kGroup];          // positions other than p*, ascending u
    double err[kGroup];
    uint8_t near_idx[kGroup];
};

inline double sqd(float u, float c)
{
    double d = static_cast<double>(u) - static_cast<double>(c);
    return d * d;
}

// Nearest centroid (ties to the lower index) for values visited in ascending order: the index
// never decreases, so one forward sweep over the ascending pattern serves the whole group.
// Plateaus of equal distance (duplicate centroids, or distances that round to the same value)
// are walked to their first entry.
inline int sweep_nearest(const float* c, float u, int j)
{
    while (j + 1 < kCentroids && sqd(u, c[j + 1]) <= sqd(u, c[j])) ++j;
    while (j > 0 && sqd(u, c[j - 1]) == sqd(u, c[j])) --j;
    return j;
}

int quantize_group(const ecco_meta& m, const uint16_t* x16, uint32_t select, float T, Scratch& s, Quantized& q)
{
    int p = 0;
    float amax = -1.0f;
    for (int i = 0; i < kGroup; ++i) {
        if ((x16[i] & 0x7fffu) >= 0x7c00u) return ECCO_ERR_NONFINITE_INPUT;
        s.x[i] = half_to_float(x16[i]);
        float a = std::fabs(s.x[i]);
        if (a > amax) { amax = a; p = i; }
    }
    q.pstar = p;
    q.qs = float_to_fp8(s.x[p] / T);
    const float scale = std::fabs(fp8_to_float(q.qs)) * T;
    int n = 0;
    for (int i = 0; i < kGroup; ++i) {
        s.u[i] = (i == p || scale == 0.0f) ? 0.0f : s.x[i] / scale;
        if (i != p) s.order[n++] = i;
    }
    int best = 0;
    if (select == ECCO_SELECT_MINMAX) {
        double lo = INFINITY, hi = -INFINITY;
        for (int i = 0; i < kGroup; ++i) {
            if (i == p) continue;
            if (s.u[i] < lo) lo = s.u[i];
            if (s.u[i] > hi) hi = s.u[i];
        }
        double best_score = INFINITY;
        for (int k = 0; k < m.S; ++k) {
            const float* c = m.pattern_f[k];
            double a = static_cast<double>(c[0]) - lo, b = static_cast<double>(c[kCentroids - 1]) - hi;
            double score = a * a + b * b;
            if (score < best_score) { best_score = score; best = k; }
        }
        std::sort(s.order, s.order + n, [&](int a, int b) { return s.u[a] < s.u[b]; });
    } else {
        std::sort(s.order, s.order + n, [&](int a, int b) { return s.u[a] < s.u[b]; });
        double best_score = INFINITY;
        for (int k = 0; k < m.S; ++k) {
            const float* c = m.pattern_f[k];
            int j = 0;
            for (int t = 0; t < n; ++t) {
                int i = s.order[t];
                j = sweep_nearest(c, s.u[i], j);
                s.err[i] = sqd(s.u[i], c[j]);
            }
            double score = 0.0;                     // summed in position order, like the definition
            for (int i = 0; i < kGroup; ++i)
                if (i != p) score += s.err[i];
            if (score < best_score) { best_score = score; best = k; }
        }
    }
    q.kp = best;
    const float* c = m.pattern_f[best];
    int j = 0;
    for (int t = 0; t < n; ++t) {
        int i = s.order[t];
        j = sweep_nearest(c, s.u[i], j);
        q.sym[i] = static_cast<uint8_t>(j);
    }
    q.sym[p] = 15;
    return ECCO_OK;
}

// ---------------------------------------------------------------------------------------------
// block writer
// ---------------------------------------------------------------------------------------------
struct BitWriter {
    uint64_t w[8] = {};
    inline void put(int pos, uint64_t v, int nbits)    // v's bit 0 goes to stream bit pos; bits past 511 dropped
    {
        if (pos >= kBlockBits) return;
        int word = pos >> 6, off = pos & 63;
        w[word] |= v << off;
        if (off + nbits > 64 && word + 1 < 8) w[word + 1] |= v >> (64 - off);
    }
};

struct GroupOut { int kp, hf, n_fit, n_pad, end_bit; };

int encode_group(const ecco_meta& m, const uint16_t* x16, uint32_t select, float T, Scratch& s, uint8_t* blk,
                 GroupOut& g, Quantized& q)
{
    int rc = quantize_group(m, x16, select, T, s, q);
    if (rc) return rc;
    // step 8: shortest total length, ties to the lower codebook id
    int total[kCodebooks] = {0, 0, 0, 0};
    for (int i = 0; i < kGroup; ++i)
        for (int h = 0; h < kCodebooks; ++h) total[h] += m.cb_len[q.kp][h][q.sym[i]];
    int hf = 0;
    for (int h = 1; h < kCodebooks; ++h)
        if (total[h] < total[hf]) hf = h;

    BitWriter bw;
    bw.put(0, q.qs, 8);
    bw.put(8, static_cast<uint64_t>(hf), 2);
    bw.put(kHeaderBits, m.kp_rev[q.kp], m.kp_len[q.kp]);
    int pos = kHeaderBits + m.kp_len[q.kp];
    const uint8_t* len = m.cb_len[q.kp][hf];
    const uint16_t* rev = m.cb_rev[q.kp][hf];
    int n_fit = 0;
    for (; n_fit < kGroup; ++n_fit) {
        int L = len[q.sym[n_fit]];
        if (pos + L > kBlockBits) {                       // step 9, clip: literal truncation at bit 512
            int room = kBlockBits - pos;
            if (room > 0) bw.put(pos, rev[q.sym[n_fit]] & ((1u << room) - 1u), room);
            break;
        }
        bw.put(pos, rev[q.sym[n_fit]], L);
        pos += L;
    }
    int n_pad = 0;
    if (n_fit == kGroup) {                                // step 9, pad: next-largest |x| first
        n_pad = std::min(kMaxPads, (kBlockBits - pos) / kPadBits);
        if (n_pad > 0) {
            int cand[kGroup], n = 0;
            for (int i = 0; i < kGroup; ++i)
                if (i != q.pstar) cand[n++] = i;
            std::partial_sort(cand, cand + n_pad, cand + n, [&](int a, int b) {
                float fa = std::fabs(s.x[a]), fb = std::fabs(s.x[b]);
                return fa > fb || (fa == fb && a < b);
            });
            for (int j = 0; j < n_pad; ++j) {
                uint64_t field = static_cast<uint64_t>(cand[j]) | (static_cast<uint64_t>(float_to_fp8(s.x[cand[j]] / T)) << 7);
                bw.put(kBlockBits - kPadBits * (j + 1), field, kPadBits);
            }
        }
    }
    std::memcpy(blk, bw.w, kBlockBytes);                  // little-endian host: stream bit k = bit k&7 of byte k>>3
    g.kp = q.kp; g.hf = hf; g.n_fit = n_fit; g.n_pad = n_pad; g.end_bit = pos;
    return ECCO_OK;
}

// ---------------------------------------------------------------------------------------------
// calibration helpers (independent, faster routes than a textbook implementation would take)
// ---------------------------------------------------------------------------------------------
struct Rng {                                             // xorshift128+
    uint64_t a, b;
    explicit Rng(uint64_t seed) : a(seed * 0x9E3779B97F4A7C15ull + 0x1234567ull), b(seed ^ 0xD1B54A32D192ED03ull)
    {
        if (!a && !b) b = 1;
        for (int i = 0; i < 8; ++i) next();
    }
    uint64_t next()
    {
        uint64_t x = a, y = b;
        a = y;
        x ^= x << 23;
        b = x ^ y ^ (x >> 17) ^ (y >> 26);
        return b + y;
    }
    double uniform() { return static_cast<double>(next() >> 11) * (1.0 / 9007199254740992.0); }
};

// step 3: 15-means of 127 sorted values by Lloyd's iteration from quantile seeds (weighted)
void group_pattern(const float* v, const float* w, int n, double* cen)
{
    for (int j = 0; j < kCentroids; ++j) cen[j] = v[std::min(n - 1, static_cast<int>((j + 0.5) * n / kCentroids))];
    for (int it = 0; it < 40; ++it) {
        double sw[kCentroids] = {}, swv[kCentroids] = {};
        int j = 0;
        for (int i = 0; i < n; ++i) {
            while (j + 1 < kCentroids && std::fabs(v[i] - cen[j + 1]) < std::fabs(v[i] - cen[j])) ++j;
            double wi = w ? w[i] : 1.0;
            sw[j] += wi;
            swv[j] += wi * v[i];
        }
        bool moved = false;
        for (int c = 0; c < kCentroids; ++c)
            if (sw[c] > 0.0) {
                double nc = swv[c] / sw[c];
                if (nc != cen[c]) { cen[c] = nc; moved = true; }
            }
        std::sort(cen, cen + kCentroids);
        if (!moved) break;
    }
}

// Lloyd's k-means with k-means++ seeding on n points of dimension d (row-major doubles)
void lloyd(const std::vector<double>& x, int n, int d, int k, uint64_t seed, int iters, std::vector<double>& cen,
           std::vector<int>& assign)
{
    Rng rng(seed);
    cen.assign(static_cast<size_t>(k) * d, 0.0);
    assign.assign(static_cast<size_t>(n), -1);
    std::vector<double> mind(static_cast<size_t>(n), INFINITY);
    auto dist = [&](int i, const double* c) {
        double s = 0.0;
        const double* p = &x[static_cast<size_t>(i) * d];
        for (int j = 0; j < d; ++j) s += (p[j] - c[j]) * (p[j] - c[j]);
        return s;
    };
    int first = std::min(n - 1, static_cast<int>(rng.uniform() * n));
    std::copy_n(&x[static_cast<size_t>(first) * d], d, cen.begin());
    for (int c = 1; c < k; ++c) {
        double tot = 0.0;
        for (int i = 0; i < n; ++i) {
            mind[i] = std::min(mind[i], dist(i, &cen[static_cast<size_t>(c - 1) * d]));
            tot += mind[i];
        }
        int pick = std::min(n - 1, static_cast<int>(rng.uniform() * n));
        if (tot > 0.0) {
            double r = rng.uniform() * tot, acc = 0.0;
            for (int i = 0; i < n; ++i) {
                acc += mind[i];
                if (acc > r) { pick = i; break; }
            }
        }
        std::copy_n(&x[static_cast<size_t>(pick) * d], d, cen.begin() + static_cast<size_t>(c) * d);
    }
    std::vector<double> sum(static_cast<size_t>(k) * d);
    std::vector<int> cnt(static_cast<size_t>(k));
    for (int it = 0; it <= iters; ++it) {
        bool changed = false;
        for (int i = 0; i < n; ++i) {
            int best = 0;
            double bd = INFINITY;
            for (int c = 0; c < k; ++c) {
                double dd = dist(i, &cen[static_cast<size_t>(c) * d]);
                if (dd < bd) { bd = dd; best = c; }
            }
            mind[i] = bd;
            if (assign[i] != best) { assign[i] = best; changed = true; }
        }
        if (!changed || it == iters) break;
        std::fill(sum.begin(), sum.end(), 0.0);
        std::fill(cnt.begin(), cnt.end(), 0);
        for (int i = 0; i < n; ++i) {
            cnt[assign[i]]++;
            for (int j = 0; j < d; ++j) sum[static_cast<size_t>(assign[i]) * d + j] += x[static_cast<size_t>(i) * d + j];
        }
        for (int c = 0; c < k; ++c) {
            if (cnt[c]) {
                for (int j = 0; j < d; ++j) cen[static_cast<size_t>(c) * d + j] = sum[static_cast<size_t>(c) * d + j] / cnt[c];
            } else {                                     // empty cluster: restart it at the worst-served point
                int far = static_cast<int>(std::max_element(mind.begin(), mind.end()) - mind.begin());
                std::copy_n(&x[static_cast<size_t>(far) * d], d, cen.begin() + static_cast<size_t>(c) * d);
                mind[far] = 0.0;
            }
        }
    }
}

// step 7: cheapest complete code over 16 symbols with all lengths in [2, 8].  Iterates over the
// number of codewords of each length; for a given multiset the sorted frequencies take the
// lengths in order.  (An explicit stack instead of recursion.)
void lengths_2_8(const double* freq, uint8_t* len)
{
    int order[kSymbols];
    std::iota(order, order + kSymbols, 0);
    std::stable_sort(order, order + kSymbols, [&](int a, int b) { return freq[a] > freq[b]; });
    double prefix[kSymbols + 1] = {0.0};
    for (int i = 0; i < kSymbols; ++i) prefix[i + 1] = prefix[i] + freq[order[i]];
    int cnt[9] = {}, best_cnt[9] = {};
    double best = INFINITY;
    // depth-first over lengths 2..7; length 8 takes what is left
    struct Frame { int L, left, kraft, c; double cost; };
    std::vector<Frame> st;
    st.push_back({2, kSymbols, 256, -1, 0.0});
    while (!st.empty()) {
        Frame& f = st.back();
        ++f.c;
        int worth = 1 << (8 - f.L);
        if (f.c > f.left || f.c * worth > f.kraft) { st.pop_back(); continue; }
        cnt[f.L] = f.c;
        int used = kSymbols - f.left;
        double cost = f.cost + (prefix[used + f.c] - prefix[used]) * f.L;
        int left = f.left - f.c, kraft = f.kraft - f.c * worth;
        if (f.L == 7) {
            if (left == kraft) {                         // the rest are 8-bit codes worth 1/256 each
                double total = cost + (prefix[kSymbols] - prefix[used + f.c]) * 8;
                if (total < best) { best = total; std::copy(cnt, cnt + 9, best_cnt); best_cnt[8] = left; }
            }
        } else {
            st.push_back({f.L + 1, left, kraft, -1, cost});
        }
    }
    int r = 0;
    for (int L = 2; L <= 8; ++L)
        for (int c = 0; c < best_cnt[L]; ++c) len[order[r++]] = static_cast<uint8_t>(L);
}

// length-limited optimal code (package-merge) for the ID_KP code; n <= 64, 2^maxlen >= n.
// Items carry a 64-bit-per-level count vector implicitly: the length of a symbol is the number
// of selected items it appears in, tracked with per-item symbol counters.
void lengths_limited(const double* freq, int n, int maxlen, uint8_t* len)
{
    struct Item { double w; std::vector<uint8_t> cnt; };
    std::vector<Item> leaves(static_cast<size_t>(n));
    for (int s = 0; s < n; ++s) {
        leaves[s].w = freq[s];
        leaves[s].cnt.assign(static_cast<size_t>(n), 0);
        leaves[s].cnt[s] = 1;
    }
    std::stable_sort(leaves.begin(), leaves.end(), [](const Item& a, const Item& b) { return a.w < b.w; });
    std::vector<Item> cur = leaves;
    for (int level = maxlen - 1; level >= 1; --level) {
        std::vector<Item> packed;
        for (size_t p = 0; p + 1 < cur.size(); p += 2) {
            Item q;
            q.w = cur[p].w + cur[p + 1].w;
            q.cnt.resize(static_cast<size_t>(n));
            for (int s = 0; s < n; ++s) q.cnt[s] = static_cast<uint8_t>(cur[p].cnt[s] + cur[p + 1].cnt[s]);
            packed.push_back(std::move(q));
        }
        std::vector<Item> merged;
        merged.reserve(packed.size() + leaves.size());
        std::merge(packed.begin(), packed.end(), leaves.begin(), leaves.end(), std::back_inserter(merged),
                   [](const Item& a, const Item& b) { return a.w < b.w; });
        cur.swap(merged);
    }
    std::fill(len, len + n, 0);
    for (int i = 0; i < 2 * n - 2; ++i)
        for (int s = 0; s < n; ++s) len[s] = static_cast<uint8_t>(len[s] + cur[i].cnt[s]);
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// C ABI: metadata
// ---------------------------------------------------------------------------------------------
extern "C" int ecco_meta_create(int32_t S, int32_t e, const uint16_t* patterns, const uint8_t* cb_len,
                                const uint8_t* kp_len, ecco_meta** out_meta)
{
    if (!patterns || !cb_len || !kp_len || !out_meta) return ECCO_ERR_INVALID_ARG;
    if (S < 2 || S > kMaxPatterns) return ECCO_ERR_BAD_META;
    ecco_meta* m = new (std::nothrow) ecco_meta();
    if (!m) return ECCO_ERR_INVALID_ARG;
    m->S = S;
    m->e = e;
    for (int k = 0; k < S; ++k) {
        std::memcpy(m->pattern[k], patterns + static_cast<size_t>(k) * kCentroids, kCentroids * 2);
        std::memcpy(m->cb_len[k], cb_len + static_cast<size_t>(k) * kCodebooks * kSymbols, kCodebooks * kSymbols);
        m->kp_len[k] = kp_len[k];
    }
    int rc = derive(m);
    if (rc) { delete m; return rc; }
    *out_meta = m;
    return ECCO_OK;
}

extern "C" int ecco_meta_get(const ecco_meta* m, int32_t* S, int32_t* e, uint16_t* patterns, uint8_t* cb_len,
                             uint8_t* kp_len)
{
    if (!m) return ECCO_ERR_INVALID_ARG;
    if (S) *S = m->S;
    if (e) *e = m->e;
    for (int k = 0; k < m->S; ++k) {
        if (patterns) std::memcpy(patterns + static_cast<size_t>(k) * kCentroids, m->pattern[k], kCentroids * 2);
        if (cb_len) std::memcpy(cb_len + static_cast<size_t>(k) * kCodebooks * kSymbols, m->cb_len[k], kCodebooks * kSymbols);
        if (kp_len) kp_len[k] = m->kp_len[k];
    }
    return ECCO_OK;
}

extern "C" void ecco_meta_free(ecco_meta* m) { delete m; }

// ---------------------------------------------------------------------------------------------
// C ABI: encoder
// ---------------------------------------------------------------------------------------------
extern "C" int ecco_encode_host(ecco_meta* m, const uint16_t* src, uint64_t n_groups, uint32_t flags, uint8_t* dst,
                                ecco_stats* stats)
{
    if (!m || (n_groups && (!src || !dst))) return ECCO_ERR_INVALID_ARG;
    if (flags & ~(ECCO_SELECT_MINMAX | ECCO_KEEP_EXPONENT)) return ECCO_ERR_INVALID_ARG;
    ensure_tables();
    if (!(flags & ECCO_KEEP_EXPONENT)) {
        int rc = fit_exponent(src, n_groups * kGroup, 0, &m->e);
        if (rc) return rc;
    }
    int rc = derive(m);
    if (rc) return rc;
    const uint32_t select = flags & ECCO_SELECT_MINMAX;
    const float T = std::ldexp(1.0f, m->e);
    const int threads = available_cores();
    std::vector<ecco_stats> part(static_cast<size_t>(threads));
    std::atomic<int> err{0};
    parallel_ranges(n_groups, threads, [&](int t, uint64_t lo, uint64_t hi) {
        Scratch s;
        Quantized q;
        GroupOut g;
        ecco_stats st;
        std::memset(&st, 0, sizeof st);
        for (uint64_t i = lo; i < hi && !err.load(std::memory_order_relaxed); ++i) {
            int r = encode_group(*m, src + i * kGroup, select, T, s, dst + i * kBlockBytes, g, q);
            if (r) { err = r; break; }
            st.n_groups++;
            if (g.n_fit < kGroup) { st.clipped_groups++; st.clipped_values += static_cast<uint64_t>(kGroup - g.n_fit); }
            if (g.n_pad) { st.padded_groups++; st.padded_values += static_cast<uint64_t>(g.n_pad); }
            st.total_bits += static_cast<uint64_t>(g.end_bit);
            st.kp_usage[g.kp]++;
            st.hf_usage[g.hf]++;
            for (int j = 0; j < kGroup; ++j) st.sym_count[q.sym[j]]++;
        }
        part[static_cast<size_t>(t)] = st;
    });
    if (err) return err;
    if (stats) {
        std::memset(stats, 0, sizeof *stats);
        for (const auto& p : part) {
            const uint64_t* a = reinterpret_cast<const uint64_t*>(&p);
            uint64_t* b = reinterpret_cast<uint64_t*>(stats);
            for (size_t i = 0; i < sizeof(ecco_stats) / 8; ++i) b[i] += a[i];
        }
    }
    return ECCO_OK;
}

// ---------------------------------------------------------------------------------------------
// C ABI: variable-length container (no clipping, no padding; groups back to back + start index)
// ---------------------------------------------------------------------------------------------
extern "C" size_t ecco_var_stream_bytes_bound(uint64_t n_groups)
{
    return static_cast<size_t>(((n_groups * kVarMaxBits + 127) / 128) * 16 + 16);
}
extern "C" size_t ecco_var_index_bytes(uint64_t n_groups)
{
    return static_cast<size_t>((8 + 8 * var_chunks(n_groups) + 4 * n_groups + 15) & ~15ull);
}

extern "C" int ecco_var_encode_host(ecco_meta* m, const uint16_t* src, uint64_t n_groups, uint32_t flags, uint8_t* dst_stream,
                                    size_t stream_capacity, void* dst_index, size_t index_capacity, uint64_t* total_bits_out)
{
    if (!m || !dst_index || (n_groups && (!src || !dst_stream))) return ECCO_ERR_INVALID_ARG;
    if (flags & ~(ECCO_SELECT_MINMAX | ECCO_KEEP_EXPONENT)) return ECCO_ERR_INVALID_ARG;
    if (index_capacity < ecco_var_index_bytes(n_groups)) return ECCO_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(dst_stream) | reinterpret_cast<uintptr_t>(dst_index)) & 7u) return ECCO_ERR_ALIGNMENT;
    ensure_tables();
    if (!(flags & ECCO_KEEP_EXPONENT)) {
        int rc = fit_exponent(src, n_groups * kGroup, 0, &m->e);
        if (rc) return rc;
    }
    int rc = derive(m);
    if (rc) return rc;
    const uint32_t select = flags & ECCO_SELECT_MINMAX;
    const float T = std::ldexp(1.0f, m->e);
    const int threads = available_cores();
    // pass 1: the bit length of every group
    std::vector<uint16_t> bits(static_cast<size_t>(n_groups));
    std::atomic<int> err{0};
    auto group_fields = [&](uint64_t g, Scratch& s, Quantized& q, int& hf) -> int {
        int r = quantize_group(*m, src + g * kGroup, select, T, s, q);
        if (r) return -1;
        int total[kCodebooks] = {0, 0, 0, 0};
        for (int i = 0; i < kGroup; ++i)
            for (int h = 0; h < kCodebooks; ++h) total[h] += m->cb_len[q.kp][h][q.sym[i]];
        hf = 0;
        for (int h = 1; h < kCodebooks; ++h)
            if (total[h] < total[hf]) hf = h;
        return kHeaderBits + m->kp_len[q.kp] + total[hf];
    };
    parallel_ranges(n_groups, threads, [&](int, uint64_t lo, uint64_t hi) {
        Scratch s;
        Quantized q;
        int hf;
        for (uint64_t g = lo; g < hi && !err.load(std::memory_order_relaxed); ++g) {
            int L = group_fields(g, s, q, hf);
            if (L < 0) { err = ECCO_ERR_NONFINITE_INPUT; break; }
            bits[g] = static_cast<uint16_t>(L);
        }
    });
    if (err) return err;
    // index
    uint64_t* idx64 = static_cast<uint64_t*>(dst_index);
    uint32_t* off32 = reinterpret_cast<uint32_t*>(idx64 + 1 + var_chunks(n_groups));
    std::vector<uint64_t> start(static_cast<size_t>(n_groups) + 1);
    uint64_t pos = 0;
    for (uint64_t g = 0; g < n_groups; ++g) {
        if ((g & ((1ull << kVarChunkShift) - 1)) == 0) idx64[1 + (g >> kVarChunkShift)] = pos;
        off32[g] = static_cast<uint32_t>(pos - idx64[1 + (g >> kVarChunkShift)]);
        start[g] = pos;
        pos += bits[g];
    }
    start[n_groups] = pos;
    idx64[0] = pos;
    if (total_bits_out) *total_bits_out = pos;
    const size_t need = static_cast<size_t>(((pos + 127) / 128) * 16);
    if (stream_capacity < need) return ECCO_ERR_INVALID_ARG;
    std::memset(dst_stream, 0, need);
    // pass 2: write the fields; neighbouring threads may share a 64-bit word at their range boundary
    uint64_t* words = reinterpret_cast<uint64_t*>(dst_stream);
    auto put = [&](uint64_t p, uint64_t v, int nbits) {
        const uint64_t w = p >> 6;
        const int off = static_cast<int>(p & 63);
        __atomic_fetch_or(&words[w], v << off, __ATOMIC_RELAXED);
        if (off + nbits > 64) __atomic_fetch_or(&words[w + 1], v >> (64 - off), __ATOMIC_RELAXED);
    };
    parallel_ranges(n_groups, threads, [&](int, uint64_t lo, uint64_t hi) {
        Scratch s;
        Quantized q;
        int hf = 0;
        for (uint64_t g = lo; g < hi; ++g) {
            group_fields(g, s, q, hf);
            uint64_t p = start[g];
            put(p, q.qs | (static_cast<uint64_t>(hf) << 8) | (static_cast<uint64_t>(m->kp_rev[q.kp]) << kHeaderBits),
                kHeaderBits + m->kp_len[q.kp]);
            p += kHeaderBits + m->kp_len[q.kp];
            for (int i = 0; i < kGroup; ++i) {
                const int L = m->cb_len[q.kp][hf][q.sym[i]];
                put(p, m->cb_rev[q.kp][hf][q.sym[i]], L);
                p += L;
            }
        }
    });
    return ECCO_OK;
}

// ---------------------------------------------------------------------------------------------
// C ABI: calibration
// ---------------------------------------------------------------------------------------------
extern "C" int ecco_calibrate_host(const uint16_t* calib, uint64_t n_groups, const float* weights,
                                   const ecco_params* p, ecco_meta** out_meta)
{
    if (!calib || !p || !out_meta) return ECCO_ERR_INVALID_ARG;
    if (p->S < 2 || p->S > kMaxPatterns || p->H != kCodebooks || p->select > ECCO_SELECT_MINMAX) return ECCO_ERR_INVALID_ARG;
    ensure_tables();
    const int S = p->S, iters = p->kmeans_iters > 0 ? p->kmeans_iters : 25;
    uint64_t use = p->max_groups ? std::min(p->max_groups, n_groups) : n_groups;
    if (use < static_cast<uint64_t>(S) || use > (1ull << 30)) return ECCO_ERR_INVALID_ARG;
    if (weights)
        for (int i = 0; i < kGroup; ++i)
            if (!(weights[i] >= 0.0f) || !std::isfinite(weights[i])) return ECCO_ERR_INVALID_ARG;
    const int n = static_cast<int>(use);
    auto group_at = [&](int i) { return calib + (n_groups * static_cast<uint64_t>(i) / use) * kGroup; };

    ecco_meta* m = new (std::nothrow) ecco_meta();
    if (!m) return ECCO_ERR_INVALID_ARG;
    m->S = S;
    int rc = fit_exponent(calib, n_groups * kGroup, p->threads, &m->e);
    if (rc) { delete m; return rc; }
    const float T = std::ldexp(1.0f, m->e);

    // steps 2-3: one ascending 15-centroid pattern per sampled group
    std::vector<double> pats(static_cast<size_t>(n) * kCentroids);
    parallel_ranges(static_cast<uint64_t>(n), p->threads, [&](int, uint64_t lo, uint64_t hi) {
        for (uint64_t g = lo; g < hi; ++g) {
            const uint16_t* x16 = group_at(static_cast<int>(g));
            float x[kGroup];
            int ps = 0;
            for (int i = 0; i < kGroup; ++i) {
                x[i] = half_to_float(x16[i]);
                if (std::fabs(x[i]) > std::fabs(x[ps])) ps = i;
            }
            float scale = std::fabs(fp8_to_float(float_to_fp8(x[ps] / T))) * T;
            std::pair<float, float> vw[kGroup - 1];
            int c = 0;
            for (int i = 0; i < kGroup; ++i)
                if (i != ps) vw[c++] = {scale == 0.0f ? 0.0f : x[i] / scale, weights ? weights[i] : 1.0f};
            std::sort(vw, vw + c);
            float v[kGroup - 1], w[kGroup - 1];
            for (int i = 0; i < c; ++i) { v[i] = vw[i].first; w[i] = vw[i].second; }
            group_pattern(v, weights ? w : nullptr, c, &pats[g * kCentroids]);
        }
    });
    // step 4: S shared patterns
    std::vector<double> cen;
    std::vector<int> assign;
    lloyd(pats, n, kCentroids, S, p->seed, iters, cen, assign);
    for (int k = 0; k < S; ++k) {
        // fp16 rounding through the float table: nearest fp16 by search over the monotone table
        for (int j = 0; j < kCentroids; ++j) {
            float c = static_cast<float>(cen[static_cast<size_t>(k) * kCentroids + j]);
            uint16_t sign = c < 0 ? 0x8000u : 0;
            float a = std::fabs(c);
            uint16_t lo = 0, hi = 0x7bff;                // largest finite
            while (lo < hi) {                            // first code with value >= a
                uint16_t mid = static_cast<uint16_t>((lo + hi) / 2);
                if (half_to_float(mid) < a) lo = static_cast<uint16_t>(mid + 1); else hi = mid;
            }
            uint16_t best = lo;
            if (lo > 0) {
                float up = half_to_float(lo) - a, dn = a - half_to_float(static_cast<uint16_t>(lo - 1));
                if (dn < up || (dn == up && ((lo - 1) & 1) == 0)) best = static_cast<uint16_t>(lo - 1);
            }
            m->pattern[k][j] = sign | best;
        }
        std::sort(m->pattern[k], m->pattern[k] + kCentroids, [](uint16_t a, uint16_t b) { return half_to_float(a) < half_to_float(b); });
    }
    // provisional complete codes so that the metadata validates while step 5 runs
    for (int k = 0; k < S; ++k) {
        m->kp_len[k] = 0;
        for (int h = 0; h < kCodebooks; ++h) std::fill(m->cb_len[k][h], m->cb_len[k][h] + kSymbols, uint8_t{4});
    }
    {
        std::vector<double> ones(static_cast<size_t>(S), 1.0);
        lengths_limited(ones.data(), S, kKpMaxLen, m->kp_len);
    }
    rc = derive(m);
    if (rc) { delete m; return rc; }

    // step 5 on the sample: pattern ids and index histograms
    std::vector<int> kp(static_cast<size_t>(n));
    std::vector<double> hist(static_cast<size_t>(n) * kSymbols, 0.0);
    std::atomic<int> err{0};
    parallel_ranges(static_cast<uint64_t>(n), p->threads, [&](int, uint64_t lo, uint64_t hi) {
        Scratch s;
        Quantized q;
        for (uint64_t g = lo; g < hi; ++g) {
            int r = quantize_group(*m, group_at(static_cast<int>(g)), p->select, T, s, q);
            if (r) { err = r; return; }
            kp[g] = q.kp;
            for (int i = 0; i < kGroup; ++i) hist[g * kSymbols + q.sym[i]] += 1.0 / kGroup;
        }
    });
    if (err) { delete m; return err; }

    // steps 6-7: H representative histograms per pattern -> H codebooks
    std::vector<double> usage(static_cast<size_t>(S), 1.0);
    for (int k = 0; k < S; ++k) {
        std::vector<double> sub;
        for (int g = 0; g < n; ++g)
            if (kp[g] == k) sub.insert(sub.end(), &hist[static_cast<size_t>(g) * kSymbols], &hist[static_cast<size_t>(g + 1) * kSymbols]);
        int cnt = static_cast<int>(sub.size() / kSymbols);
        usage[k] += cnt;
        std::vector<double> rep(static_cast<size_t>(kCodebooks) * kSymbols, 1.0 / kSymbols);
        if (cnt >= kCodebooks) {
            std::vector<int> a;
            lloyd(sub, cnt, kSymbols, kCodebooks, p->seed + 1 + static_cast<uint64_t>(k), iters, rep, a);
        } else if (cnt > 0) {
            for (int s = 0; s < kSymbols; ++s) {
                double mean = 0.0;
                for (int g = 0; g < cnt; ++g) mean += sub[static_cast<size_t>(g) * kSymbols + s];
                for (int h = 0; h < kCodebooks; ++h) rep[static_cast<size_t>(h) * kSymbols + s] = mean / cnt;
            }
        }
        for (int h = 0; h < kCodebooks; ++h) lengths_2_8(&rep[static_cast<size_t>(h) * kSymbols], m->cb_len[k][h]);
    }
    lengths_limited(usage.data(), S, kKpMaxLen, m->kp_len);
    rc = derive(m);
    if (rc) { delete m; return rc; }
    *out_meta = m;
    return ECCO_OK;
}

// ---------------------------------------------------------------------------------------------
// C ABI: device image
// ---------------------------------------------------------------------------------------------
namespace {

// code shapes of a metadata set and the plan of its decode tables
struct ImagePlan {
    int n_shapes = 0;
    uint8_t counts[kMaxShapes][kMaxLen + 1] = {};          // shape -> number of codewords per length
    int shape_of[kMaxPatterns][kCodebooks] = {};
    int width[kMaxShapes] = {};                            // pair-table index bits per shape, 0 = none
    uint32_t pair_off[kMaxShapes] = {};                    // byte offset of the shape's pair table in the pair region
    uint32_t pair_bytes = 0, pair_align = 0;
    uint32_t total_bytes = 0, off_pair = 0;
};

// probability that two consecutive codewords of the shape do not both end within W bits, symbols drawn with
// probability 2^-length (what the code is optimal for)
double escape_rate(const uint8_t* counts, int W)
{
    double esc = 0.0;
    for (int l0 = kMinLen; l0 <= kMaxLen; ++l0)
        for (int l1 = kMinLen; l1 <= kMaxLen; ++l1)
            if (l0 + l1 > W) esc += std::ldexp(static_cast<double>(counts[l0]), -l0) * std::ldexp(static_cast<double>(counts[l1]), -l1);
    return esc;
}

void plan_image(const ecco_meta& m, ImagePlan& p)
{
    // Expected use of a shape: what the ID_KP code lengths say about its patterns (a pattern coded in L bits is
    // used about 2^-L of the time), the four codebooks of a pattern alike.  A function of the metadata alone, so
    // that tensors encoded with the same patterns and codebooks get the same tables, hence the same table hash.
    double use[kMaxShapes] = {};
    for (int k = 0; k < kMaxPatterns; ++k)
        for (int h = 0; h < kCodebooks; ++h) {
            uint8_t c[kMaxLen + 1] = {};
            if (k < m.S) for (int s = 0; s < kSymbols; ++s) ++c[m.cb_len[k][h][s]];
            else c[4] = kSymbols;                          // rows of unused patterns decode as sixteen 4-bit codewords
            int id = -1;
            for (int i = 0; i < p.n_shapes && id < 0; ++i)
                if (!std::memcmp(p.counts[i], c, sizeof c)) id = i;
            if (id < 0) { id = p.n_shapes++; std::memcpy(p.counts[id], c, sizeof c); }
            p.shape_of[k][h] = id;
            if (k < m.S) use[id] += std::ldexp(1.0, -m.kp_len[k]) / kCodebooks;
        }
    // widths: everyone starts at the minimum; then the upgrade that removes the most escapes per byte, while it fits
    uint32_t bytes = static_cast<uint32_t>(p.n_shapes) * (2u << kPairMinBits);
    if (bytes <= kPairBudgetBytes) {
        for (int i = 0; i < p.n_shapes; ++i) p.width[i] = kPairMinBits;
        for (;;) {
            int best = -1;
            double best_gain = 0.0;
            for (int i = 0; i < p.n_shapes; ++i) {
                const int W = p.width[i];
                if (W >= kPairMaxBits || bytes + (2u << W) > kPairBudgetBytes) continue;
                const double gain = (use[i] + 1e-9) * (escape_rate(p.counts[i], W) - escape_rate(p.counts[i], W + 1)) / static_cast<double>(2u << W);
                if (best < 0 || gain > best_gain) { best = i; best_gain = gain; }
            }
            if (best < 0 || best_gain <= 0.0) break;
            bytes += 2u << p.width[best];
            ++p.width[best];
        }
        uint32_t off = 0;
        for (int W = kPairMaxBits; W >= kPairMinBits; --W)      // widest first: every table starts at a multiple of its size
            for (int i = 0; i < p.n_shapes; ++i)
                if (p.width[i] == W) { p.pair_off[i] = off; off += 2u << W; if (!p.pair_align) p.pair_align = 2u << W; }
        p.pair_bytes = off;
    }
    p.off_pair = (kOffShapeLut + static_cast<uint32_t>(p.n_shapes) * 256u + 15u) & ~15u;
    p.total_bytes = p.off_pair + p.pair_bytes;
}

inline uint64_t fnv1a(const uint8_t* b, size_t n, uint64_t h)
{
    for (size_t i = 0; i < n; ++i) { h ^= b[i]; h *= 1099511628211ull; }
    return h;
}

}  // namespace

extern "C" size_t ecco_meta_device_bytes(const ecco_meta* m)
{
    if (!m) return 0;
    ecco_meta tmp = *m;
    if (derive(&tmp)) return 0;
    ImagePlan* p = new ImagePlan;
    plan_image(tmp, *p);
    const size_t n = p->total_bytes;
    delete p;
    return n;
}

extern "C" int ecco_meta_serialize_device(const ecco_meta* m, void* host_staging, size_t bytes)
{
    if (!m || !host_staging) return ECCO_ERR_INVALID_ARG;
    ecco_meta tmp = *m;
    int rc = derive(&tmp);
    if (rc) return rc;
    std::unique_ptr<ImagePlan> plan(new ImagePlan);
    ImagePlan& p = *plan;
    plan_image(tmp, p);
    if (bytes < p.total_bytes) return ECCO_ERR_INVALID_ARG;
    uint8_t* base = static_cast<uint8_t*>(host_staging);
    std::memset(base, 0, p.total_bytes);
    std::memcpy(base + kOffPattern, tmp.pattern, kPatternBytes);
    // ID_KP table: every 12-bit window whose low kp_len bits equal the reversed codeword
    uint16_t* kpl = reinterpret_cast<uint16_t*>(base + kOffKpLut);
    for (int k = 0; k < tmp.S; ++k) {
        int L = tmp.kp_len[k];
        for (uint32_t hi = 0; hi < (1u << (kKpMaxLen - L)); ++hi)
            kpl[tmp.kp_rev[k] | (hi << L)] = static_cast<uint16_t>(k | (L << 8));
    }
    // encoder tables: codeword in stream order (first code bit in bit 0) and its length
    uint16_t* ecb = reinterpret_cast<uint16_t*>(base + kOffEncCb);
    uint16_t* ekp = reinterpret_cast<uint16_t*>(base + kOffEncKp);
    for (int k = 0; k < tmp.S; ++k) {
        ekp[k] = static_cast<uint16_t>(tmp.kp_rev[k] | (tmp.kp_len[k] << 12));
        for (int c = 0; c < kCodebooks; ++c)
            for (int s = 0; s < kSymbols; ++s)
                ecb[(static_cast<size_t>(k) * kCodebooks + c) * kSymbols + s] =
                    static_cast<uint16_t>(tmp.cb_rev[k][c][s] | (tmp.cb_len[k][c][s] << 8));
    }
    // codebook records: shape, pair table, symbol -> rank (rank = position in (length, symbol id) order)
    uint32_t* rec = reinterpret_cast<uint32_t*>(base + kOffCbRec);
    for (int k = 0; k < kMaxPatterns; ++k)
        for (int c = 0; c < kCodebooks; ++c) {
            const int sh = p.shape_of[k][c];
            uint64_t rank_of = 0;
            int rank = 0;
            for (int L = kMinLen; L <= kMaxLen; ++L)
                for (int s = 0; s < kSymbols; ++s)
                    if ((k < tmp.S ? tmp.cb_len[k][c][s] : 4) == L) rank_of |= static_cast<uint64_t>(rank++) << (4 * s);
            uint32_t* r = rec + (static_cast<size_t>(k) * kCodebooks + c) * 4;
            r[0] = (p.pair_off[sh] >> 9) | (static_cast<uint32_t>(sh) << 8) | (static_cast<uint32_t>(p.width[sh]) << 16);
            r[1] = 0;
            r[2] = static_cast<uint32_t>(rank_of);
            r[3] = static_cast<uint32_t>(rank_of >> 32);
        }
    // shape tables, then pair tables built from them
    for (int sh = 0; sh < p.n_shapes; ++sh) {
        uint8_t t[256];                                    // the shape table in natural order
        uint32_t code = 0;
        int rank = 0;
        for (int L = kMinLen; L <= kMaxLen; ++L) {
            for (int i = 0; i < p.counts[sh][L]; ++i, ++code, ++rank) {
                const uint32_t rev = bit_reverse(code, L);
                for (uint32_t hi = 0; hi < (1u << (kMaxLen - L)); ++hi) t[rev | (hi << L)] = static_cast<uint8_t>((L << 4) | rank);
            }
            code <<= 1;
        }
        const uint32_t rot = table_rotation(static_cast<uint32_t>(sh));
        uint8_t* st = base + kOffShapeLut + static_cast<size_t>(sh) * 256;
        for (uint32_t i = 0; i < 256; ++i) st[i ^ rot] = t[i];
        const int W = p.width[sh];
        if (!W) continue;
        uint16_t* pt = reinterpret_cast<uint16_t*>(base + p.off_pair + p.pair_off[sh]);
        for (uint32_t idx = 0; idx < (1u << W); ++idx) {
            const uint32_t e0 = t[idx & 255u], l0 = e0 >> 4, r0 = e0 & 15u;
            const uint32_t room = static_cast<uint32_t>(W) - l0;              // bits of the window after the first codeword
            const uint32_t e1 = t[(idx >> l0) & 255u], l1 = e1 >> 4, r1 = e1 & 15u;   // bits past the window read as zero
            // a codeword no longer than the bits on hand is fully inside them, so it is the real one
            pt[idx ^ (rot >> 1)] = l1 <= room ? static_cast<uint16_t>((l0 + l1) | (r0 << 7) | (r1 << 11))
                                              : static_cast<uint16_t>(l0 | (r0 << 7) | 0x8000u);
        }
    }
    DevHeader h;
    std::memset(&h, 0, sizeof h);
    h.magic = kDevMagic; h.version = kDevVersion; h.S = tmp.S; h.H = kCodebooks; h.e = tmp.e;
    h.T = std::ldexp(1.0f, tmp.e);
    h.total_bytes = p.total_bytes;
    h.n_shapes = static_cast<uint32_t>(p.n_shapes);
    h.shape_bytes = static_cast<uint32_t>(p.n_shapes) * 256u;
    h.pair_bytes = p.pair_bytes;
    h.pair_align = p.pair_align;
    h.off_pair = p.off_pair;
    uint64_t hash = 1469598103934665603ull;
    hash = fnv1a(base + kOffPattern, kFixedTableBytes, hash);
    hash = fnv1a(base + kOffShapeLut, p.total_bytes - kOffShapeLut, hash);
    h.hash_lo = static_cast<uint32_t>(hash);
    h.hash_hi = static_cast<uint32_t>(hash >> 32);
    std::memcpy(base, &h, sizeof h);
    return ECCO_OK;
}

extern "C" const char* ecco_error_string(int code)
{
    switch (code) {
        case ECCO_OK: return "ok";
        case ECCO_ERR_INVALID_ARG: return "invalid argument";
        case ECCO_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case ECCO_ERR_NONFINITE_INPUT: return "non-finite input value";
        case ECCO_ERR_BAD_META: return "inconsistent metadata";
        case ECCO_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x";
        case ECCO_ERR_CUDA: return "CUDA error (see ecco_last_cuda_error)";
        case ECCO_ERR_WORKSPACE: return "workspace too small";
        case ECCO_ERR_DEVICE_TIMEOUT: return "a device-side bounded wait expired";
        default: return "unknown error";
    }
}
