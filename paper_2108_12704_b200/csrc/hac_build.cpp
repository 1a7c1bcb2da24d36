// Host-side format builder: pruning (Sect. III-B), weight sharing (Sect. III-C.1, III-C.3),
// Huffman code and the HAC / sHAC layouts (Sect. IV-B, IV-C), plus the offset index and the
// decoding tables the kernels use.  One-off work per layer; everything here is integer or fp64
// and must reproduce the format bit for bit on every run.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <new>
#include <numeric>

#include "hac_internal.h"

namespace hacb200 {

namespace {

// SplitMix64 (Steele, Lea, Flood, OOPSLA 2014) as a counter-based generator: draw i mixes
// seed + (i + 1) * golden-ratio increment.
inline uint64_t splitmix64_at(uint64_t seed, uint64_t i) {
    uint64_t z = seed + (i + 1) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

struct Shared {                      // result of weight sharing over the q non-null weights
    std::vector<float> level_value;  // value of each level (not yet merged / sorted)
    std::vector<uint32_t> level_of;  // [q] level of each weight, column-major order
};

// Sect. III-C.1: Lloyd's k-means on scalars.  Centroids stay sorted, so the nearest centroid of w
// is found by counting the midpoints below w; sums run in storage order in fp64.
int share_kmeans(const std::vector<double>& data, uint32_t k, uint32_t iters, uint64_t seed,
                 Shared& out) {
    const size_t q = data.size();
    std::vector<double> distinct(data);
    std::sort(distinct.begin(), distinct.end());
    distinct.erase(std::unique(distinct.begin(), distinct.end()), distinct.end());
    out.level_of.resize(q);
    if (distinct.size() <= k) {      // fewer distinct values than clusters: they are the codebook
        out.level_value.resize(distinct.size());
        for (size_t l = 0; l < distinct.size(); ++l) out.level_value[l] = (float)distinct[l];
        for (size_t p = 0; p < q; ++p)
            out.level_of[p] = (uint32_t)(std::lower_bound(distinct.begin(), distinct.end(), data[p]) -
                                         distinct.begin());
        return HAC_OK;
    }
    // seeded start: partial Fisher-Yates over the distinct values
    std::vector<double> centroid(k);
    {
        const uint64_t U = distinct.size();
        std::vector<uint32_t> perm(U);
        std::iota(perm.begin(), perm.end(), 0u);
        for (uint64_t i = 0; i < k; ++i) {
            uint64_t j = i + splitmix64_at(seed, i) % (U - i);
            std::swap(perm[i], perm[j]);
            centroid[i] = distinct[perm[i]];
        }
        std::sort(centroid.begin(), centroid.end());
    }
    std::vector<double>().swap(distinct);
    std::vector<double> mid(k > 1 ? k - 1 : 0), acc(k);
    std::vector<int64_t> members(k);
    for (uint32_t it = 0;; ++it) {
        for (uint32_t l = 0; l + 1 < k; ++l) mid[l] = (centroid[l] + centroid[l + 1]) * 0.5;
        std::fill(acc.begin(), acc.end(), 0.0);
        std::fill(members.begin(), members.end(), (int64_t)0);
        const double* mb = mid.data();
        const double* me = mb + mid.size();
        for (size_t p = 0; p < q; ++p) {
            const double w = data[p];
            const uint32_t l = (uint32_t)(std::lower_bound(mb, me, w) - mb);   // #midpoints < w
            out.level_of[p] = l;
            acc[l] += w;
            members[l] += 1;
        }
        if (it == iters) break;
        for (uint32_t l = 0; l < k; ++l)
            if (members[l] > 0) centroid[l] = acc[l] / (double)members[l];
        std::sort(centroid.begin(), centroid.end());
    }
    out.level_value.resize(k);
    for (uint32_t l = 0; l < k; ++l) out.level_value[l] = (float)centroid[l];
    return HAC_OK;
}

// Sect. III-C.3: uniform grid of k levels laid over [min, max] of the non-null weights.
int share_uniform(const std::vector<double>& data, uint32_t k, Shared& out) {
    const size_t q = data.size();
    double lo = data[0], hi = data[0];
    for (size_t p = 1; p < q; ++p) { lo = std::min(lo, data[p]); hi = std::max(hi, data[p]); }
    out.level_of.assign(q, 0u);
    if (hi == lo) { out.level_value.assign(1, (float)lo); return HAC_OK; }
    const double delta = (hi - lo) / (double)(k - 1);
    out.level_value.resize(k);
    for (uint32_t l = 0; l < k; ++l) {
        volatile double step = (double)l * delta;      // product rounded on its own (no fused add)
        out.level_value[l] = (float)(lo + step);
    }
    const double top = (double)(k - 1);
    for (size_t p = 0; p < q; ++p) {
        double t = std::floor((data[p] - lo) / delta + 0.5);
        if (t < 0.0) t = 0.0;
        if (t > top) t = top;
        out.level_of[p] = (uint32_t)t;
    }
    return HAC_OK;
}

int share_none(const std::vector<double>& data, Shared& out);

// Sect. III-C.3 as printed, with d = 0: w = delta * round(w / delta) (rounding half up).  delta is tuned
// to the number of values wanted (the paper's setting for uUQ): 70 halvings of [0, 4 max|w|]; a trial
// delta that leaves at most k distinct levels becomes the upper end, and the upper end is used.
int share_grid(const std::vector<double>& data, uint32_t k, Shared& out) {
    const size_t q = data.size();
    {
        std::vector<double> distinct(data);
        std::sort(distinct.begin(), distinct.end());
        distinct.erase(std::unique(distinct.begin(), distinct.end()), distinct.end());
        if (distinct.size() <= k) return share_none(data, out);
    }
    double amax = 0.0;
    for (size_t p = 0; p < q; ++p) amax = std::max(amax, std::fabs(data[p]));
    std::vector<int64_t> lev(q);
    std::vector<unsigned char> seen;
    // number of distinct levels at `delta`; stops counting once it exceeds `limit`
    auto distinct_levels = [&](double delta, uint64_t limit) -> uint64_t {
        int64_t lo = INT64_MAX, hi = INT64_MIN;
        for (size_t p = 0; p < q; ++p) {
            const double t = std::floor(data[p] / delta + 0.5);
            if (!(std::fabs(t) < 9.0e18)) return limit + 1;          // delta far too small
            lev[p] = (int64_t)t;
            lo = std::min(lo, lev[p]); hi = std::max(hi, lev[p]);
        }
        const uint64_t span = (uint64_t)(hi - lo) + 1;
        if (span <= ((uint64_t)1 << 26)) {
            seen.assign(span, 0);
            uint64_t count = 0;
            for (size_t p = 0; p < q; ++p) {
                unsigned char& s = seen[(size_t)(lev[p] - lo)];
                if (!s) { s = 1; if (++count > limit) return count; }
            }
            return count;
        }
        std::vector<int64_t> sorted(lev);
        std::sort(sorted.begin(), sorted.end());
        return (uint64_t)(std::unique(sorted.begin(), sorted.end()) - sorted.begin());
    };
    double a = 0.0, b = 4.0 * amax;
    for (int it = 0; it < 70; ++it) {
        const double mid = 0.5 * (a + b);
        if (distinct_levels(mid, k) <= k) b = mid; else a = mid;
    }
    const double delta = b;
    int64_t lo = INT64_MAX, hi = INT64_MIN;
    for (size_t p = 0; p < q; ++p) {
        lev[p] = (int64_t)std::floor(data[p] / delta + 0.5);
        lo = std::min(lo, lev[p]); hi = std::max(hi, lev[p]);
    }
    const uint64_t span = (uint64_t)(hi - lo) + 1;
    if (span > ((uint64_t)1 << 26)) return HAC_ERR_K_TOO_LARGE;
    out.level_value.resize(span);
    for (uint64_t l = 0; l < span; ++l) {
        volatile double v = (double)(lo + (int64_t)l) * delta;
        out.level_value[l] = (float)v;
    }
    out.level_of.resize(q);
    for (size_t p = 0; p < q; ++p) out.level_of[p] = (uint32_t)(lev[p] - lo);
    return HAC_OK;
}

// Sect. III-C.2 (PWS): k representatives at the i/(k-1) quantiles (order statistics of the sorted
// weights); a weight between two neighbouring ones becomes the upper one with probability
// (w - lo)/(hi - lo), else the lower one.  One uniform number per weight, from its position.
int share_pws(const std::vector<double>& data, uint32_t k, uint64_t seed, Shared& out) {
    const size_t q = data.size();
    std::vector<double> srt(data);
    std::sort(srt.begin(), srt.end());
    {
        std::vector<double> distinct(srt);
        distinct.erase(std::unique(distinct.begin(), distinct.end()), distinct.end());
        if (distinct.size() <= k) return share_none(data, out);
    }
    std::vector<double> ext(k);
    for (uint32_t i = 0; i < k; ++i) ext[i] = srt[(size_t)(((uint64_t)i * (uint64_t)(q - 1)) / (uint64_t)(k - 1))];
    ext.erase(std::unique(ext.begin(), ext.end()), ext.end());
    std::vector<double>().swap(srt);
    const size_t r = ext.size();
    out.level_value.resize(r);
    for (size_t l = 0; l < r; ++l) out.level_value[l] = (float)ext[l];
    out.level_of.resize(q);
    for (size_t p = 0; p < q; ++p) {
        const double w = data[p];
        size_t j = (size_t)(std::upper_bound(ext.begin(), ext.end(), w) - ext.begin());    // extremes <= w
        j = j == 0 ? 0 : j - 1;
        if (j > r - 2) j = r - 2;
        const double p_hi = (w - ext[j]) / (ext[j + 1] - ext[j]);
        const double u = (double)(splitmix64_at(seed, (uint64_t)p) >> 11) * 0x1.0p-53;
        out.level_of[p] = (uint32_t)(u < p_hi ? j + 1 : j);
    }
    return HAC_OK;
}

int share_none(const std::vector<double>& data, Shared& out) {
    std::vector<double> distinct(data);
    std::sort(distinct.begin(), distinct.end());
    distinct.erase(std::unique(distinct.begin(), distinct.end()), distinct.end());
    if (distinct.size() > HAC_MAX_SYMBOLS) return HAC_ERR_K_TOO_LARGE;
    out.level_value.resize(distinct.size());
    for (size_t l = 0; l < distinct.size(); ++l) out.level_value[l] = (float)distinct[l];
    out.level_of.resize(data.size());
    for (size_t p = 0; p < data.size(); ++p)
        out.level_of[p] = (uint32_t)(std::lower_bound(distinct.begin(), distinct.end(), data[p]) -
                                     distinct.begin());
    return HAC_OK;
}

// Huffman code lengths (Sect. IV-B) with the two-queue method: leaves in (count, id) order, merged
// nodes in creation order, a leaf taken before a merged node of equal weight.
int huffman_code_lengths(const std::vector<int64_t>& counts, std::vector<uint8_t>& len) {
    const uint32_t k = (uint32_t)counts.size();
    len.assign(k, 0);
    if (k == 0) return HAC_OK;
    if (k == 1) { len[0] = 1; return HAC_OK; }
    std::vector<uint32_t> order(k);
    std::iota(order.begin(), order.end(), 0u);
    std::stable_sort(order.begin(), order.end(),
                     [&](uint32_t a, uint32_t b) { return counts[a] < counts[b]; });
    // nodes 0..k-1: leaves in sorted order; k..2k-2: merged nodes in creation order
    std::vector<int64_t> weight(2 * k - 1);
    std::vector<uint32_t> up(2 * k - 1, 0);
    for (uint32_t i = 0; i < k; ++i) weight[i] = counts[order[i]];
    uint32_t leaf = 0, inner = k, made = k;
    auto pop = [&]() -> uint32_t {
        if (leaf < k && (inner >= made || weight[leaf] <= weight[inner])) return leaf++;
        return inner++;
    };
    while (made < 2 * k - 1) {
        uint32_t a = pop();
        uint32_t b = pop();
        weight[made] = weight[a] + weight[b];
        up[a] = made; up[b] = made;
        ++made;
    }
    std::vector<uint32_t> depth(2 * k - 1, 0);
    for (int64_t v = (int64_t)2 * k - 3; v >= 0; --v) depth[v] = depth[up[v]] + 1;
    for (uint32_t i = 0; i < k; ++i) {
        if (depth[i] > (uint32_t)kMaxCodeLen) return HAC_ERR_CODE_TOO_LONG;
        len[order[i]] = (uint8_t)depth[i];
    }
    return HAC_OK;
}

// Canonical assignment: count the code words of each length, give each length its first code
// (previous first + previous count, doubled), then hand codes out in symbol-id order per length.
void canonical_assign(const std::vector<uint8_t>& len, std::vector<uint32_t>& codes) {
    uint32_t per_len[kMaxCodeLen + 2] = {0};
    for (uint8_t l : len) per_len[l]++;
    uint64_t next[kMaxCodeLen + 2] = {0};
    uint64_t code = 0;
    for (int l = 1; l <= kMaxCodeLen; ++l) {
        code = (code + per_len[l - 1]) << 1;
        next[l] = code;
    }
    codes.resize(len.size());
    for (size_t s = 0; s < len.size(); ++s) codes[s] = (uint32_t)next[len[s]]++;
}

struct BitWriter {
    std::vector<uint32_t>& words;
    uint64_t acc = 0;     // pending bits, right aligned
    int pending = 0;
    int64_t total = 0;
    explicit BitWriter(std::vector<uint32_t>& w) : words(w) {}
    inline void put(uint32_t code, int len) {
        acc = (acc << len) | code;
        pending += len;
        total += len;
        if (pending >= 32) {
            pending -= 32;
            words.push_back((uint32_t)(acc >> pending));
        }
    }
    void finish() {
        if (pending > 0) words.push_back((uint32_t)(acc << (32 - pending)));
        pending = 0;
    }
};

}  // namespace

void make_decode_tables(Format& f) {
    DecodeTables& t = f.tables;
    const uint32_t k = (uint32_t)f.codebook.size();
    t = DecodeTables();
    if (k == 0) { t.lut_bits = 1; t.lut.assign(2, 0); t.l1_bits = 1; t.l1.assign(4, 0u); return; }
    std::vector<uint32_t> by_rank(k);
    std::iota(by_rank.begin(), by_rank.end(), 0u);
    std::stable_sort(by_rank.begin(), by_rank.end(),
                     [&](uint32_t a, uint32_t b) { return f.code_len[a] < f.code_len[b]; });
    t.rank_value.resize(k);
    t.rank_symbol.resize(k);
    for (uint32_t r = 0; r < k; ++r) {
        t.rank_value[r] = f.codebook[by_rank[r]];
        t.rank_symbol[r] = (uint16_t)by_rank[r];
    }
    t.lut_bits = std::min<int>((int)f.max_len, kLutBitsMax);
    t.lut.assign((size_t)1 << t.lut_bits, 0);
    uint32_t per_len[kMaxCodeLen + 2] = {0};
    for (uint32_t s = 0; s < k; ++s) per_len[f.code_len[s]]++;
    uint32_t rank = 0;
    uint64_t first = 0;                      // first code of the current length
    for (int l = 1; l <= kMaxCodeLen; ++l) {
        first = (l == 1) ? 0 : (first + per_len[l - 1]) << 1;
        t.first_left[l] = (uint32_t)(first << (32 - l));
        t.rank_base[l] = rank;
        t.limit[l] = (first + per_len[l]) << (32 - l);
        rank += per_len[l];
    }
    t.limit[kMaxCodeLen + 1] = (uint64_t)1 << 32;
    for (uint32_t r = 0; r < k; ++r) {
        const uint32_t s = by_rank[r];
        const int l = f.code_len[s];
        if (l > t.lut_bits) continue;
        const uint32_t lo = f.codes[s] << (t.lut_bits - l);
        const uint32_t span = 1u << (t.lut_bits - l);
        const uint16_t e = (uint16_t)((r << 4) | (uint32_t)l);      // l <= kLutBitsMax = 12, r < 4096
        for (uint32_t i = 0; i < span; ++i) t.lut[lo + i] = e;
    }
    // two-level table: direct entries for code words of at most l1_bits bits, sub-tables behind
    // the prefixes that longer code words share
    auto bits_of = [](float v) { uint32_t b; std::memcpy(&b, &v, 4); return b; };
    t.l1_bits = std::min<int>((int)f.max_len, kL1BitsMax);
    const uint32_t L1 = (uint32_t)t.l1_bits;
    for (int sub_max = kSubBitsMax; sub_max >= 1; --sub_max) {
        t.l1.assign((size_t)2 << L1, 0u);
        t.sub.clear();
        std::vector<uint32_t> longest((size_t)1 << L1, 0u);    // longest code word behind each prefix
        for (uint32_t s = 0; s < k; ++s) {
            const uint32_t l = f.code_len[s];
            if (l <= L1) {
                const uint32_t lo = f.codes[s] << (L1 - l), span = 1u << (L1 - l);
                for (uint32_t i = 0; i < span; ++i) { t.l1[2 * (lo + i)] = bits_of(f.codebook[s]); t.l1[2 * (lo + i) + 1] = l; }
            } else {
                const uint32_t pre = f.codes[s] >> (l - L1);
                longest[pre] = std::max(longest[pre], l);
            }
        }
        std::vector<uint32_t> sub_base((size_t)1 << L1, 0u), sub_bits((size_t)1 << L1, 0u);
        for (uint32_t pre = 0; pre < (1u << L1); ++pre) {
            if (longest[pre] == 0) continue;
            const uint32_t b = std::min<uint32_t>(longest[pre] - L1, (uint32_t)sub_max);
            sub_base[pre] = (uint32_t)(t.sub.size() / 2);
            sub_bits[pre] = b;
            t.sub.resize(t.sub.size() + ((size_t)2 << b), 0u);
            t.l1[2 * pre] = sub_base[pre] * 8u;
            t.l1[2 * pre + 1] = 0x80000000u | b;
        }
        for (uint32_t s = 0; s < k; ++s) {
            const uint32_t l = f.code_len[s];
            if (l <= L1) continue;
            const uint32_t pre = f.codes[s] >> (l - L1), b = sub_bits[pre];
            if (l > L1 + b) continue;                          // left to the search over lengths
            const uint32_t rem = f.codes[s] & ((1u << (l - L1)) - 1u);
            const uint32_t lo = rem << (L1 + b - l), span = 1u << (L1 + b - l);
            for (uint32_t i = 0; i < span; ++i) {
                t.sub[2 * (sub_base[pre] + lo + i)] = bits_of(f.codebook[s]);
                t.sub[2 * (sub_base[pre] + lo + i) + 1] = l;
            }
        }
        if (t.sub.size() * 4 <= kSubTableBytesMax) break;
    }
    // magnitude table: only when the prefix table leaves code words to the sub-tables
    double long_count = 0.0;
    for (uint32_t s = 0; s < k; ++s)
        if (f.code_len[s] > L1) long_count += (double)f.counts[s];
    t.l1_unresolved = f.symbols ? long_count / (double)f.symbols : 0.0;
    t.xt_mant = -1;
    t.xt.clear();
    t.use_xt = false;
    if (t.l1_unresolved > 0.0) {
        for (int mant = 3; mant <= kXtMantMax; ++mant) {
            std::vector<uint32_t> xt((size_t)64 << mant, 0u);
            for (size_t c = 0; c < ((size_t)32 << mant); ++c) xt[2 * c + 1] = 0x80000000u;
            double unresolved = 0.0;
            for (uint32_t s = 0; s < k; ++s) {
                const uint32_t l = f.code_len[s];
                const uint32_t lo = l >= 32 ? f.codes[s] : f.codes[s] << (32 - l);
                const uint32_t hi = l >= 32 ? lo : lo + ((1u << (32 - l)) - 1u);
                const uint32_t ia = xt_index(lo, mant), ib = xt_index(hi, mant);     // ia >= ib
                const bool a_inside = lo == 0u || xt_index(lo - 1u, mant) != ia;
                const bool b_inside = hi == 0xffffffffu || xt_index(hi + 1u, mant) != ib;
                auto put = [&](uint32_t c) { xt[2 * c] = bits_of(f.codebook[s]); xt[2 * c + 1] = l; };
                for (uint32_t c = ib + 1; c < ia; ++c) put(c);
                if (ia == ib) { if (a_inside && b_inside) put(ia); }
                else { if (a_inside) put(ia); if (b_inside) put(ib); }
                // share of this code word's range that falls into cells shared with a neighbour
                // (taken as uniform over the range): walk inwards from both ends
                double bad = 0.0;
                const double range = (double)hi - (double)lo + 1.0;
                if (!(ia == ib ? (a_inside && b_inside) : a_inside)) {
                    uint32_t end = lo;                     // last window of cell ia inside the range (binary search)
                    uint32_t a = lo, b = hi;
                    while (a < b) { const uint32_t mid = a + (b - a + 1) / 2; if (xt_index(mid, mant) == ia) a = mid; else b = mid - 1; }
                    end = a;
                    bad += (double)end - (double)lo + 1.0;
                }
                if (ia != ib && !b_inside) {
                    uint32_t a = lo, b = hi;               // first window of cell ib inside the range
                    while (a < b) { const uint32_t mid = a + (b - a) / 2; if (xt_index(mid, mant) == ib) b = mid; else a = mid + 1; }
                    bad += (double)hi - (double)a + 1.0;
                }
                unresolved += (double)f.counts[s] * std::min(1.0, bad / range);
            }
            unresolved = f.symbols ? unresolved / (double)f.symbols : 0.0;
            if (t.xt_mant < 0 || unresolved < t.xt_unresolved) {
                t.xt_mant = mant; t.xt.swap(xt); t.xt_unresolved = unresolved;
            }
            if (t.xt_unresolved == 0.0) break;
        }
        t.use_xt = t.xt_unresolved < t.l1_unresolved;
        if (!t.use_xt) { t.xt.clear(); t.xt_mant = -1; }
    }
    // zero-run table: for streams that are mostly 1-bit zero code words
    t.l1_runs.clear();
    t.zero_len = 0;
    double zero_share = 0.0;
    if (!f.sparse) {
        for (uint32_t s = 0; s < k; ++s)
            if (f.codebook[s] == 0.0f) {
                t.zero_len = f.code_len[s];
                zero_share = f.symbols ? (double)f.counts[s] / (double)f.symbols : 0.0;
            }
    }
    // (measured: a gain from about 90 % zeros on; below that the plain table is as fast or faster)
    if (t.zero_len == 1 && zero_share >= 0.9 && t.zero_len < L1) {
        const uint32_t zero_bits = bits_of(0.0f);
        t.l1_runs.assign((size_t)2 << L1, 0u);
        const uint32_t mask = (1u << L1) - 1u;
        for (uint32_t idx = 0; idx < (1u << L1); ++idx) {
            uint32_t pos = 0, covered = 0, value = zero_bits;
            while (covered < 200) {
                const uint32_t at = (idx << pos) & mask;            // the remaining bits, left aligned
                const uint32_t v = t.l1[2 * at], meta = t.l1[2 * at + 1];
                if ((meta & 0x80000000u) || meta == 0 || meta > L1 - pos) break;   // does not end inside the prefix
                pos += meta;
                ++covered;
                if (v != zero_bits) { value = v; break; }
                if (pos >= L1) break;
            }
            if (covered == 0) {                                     // a single long code word: keep the entry
                t.l1_runs[2 * idx] = t.l1[2 * idx];
                t.l1_runs[2 * idx + 1] = t.l1[2 * idx + 1];
            } else {
                t.l1_runs[2 * idx] = value;
                t.l1_runs[2 * idx + 1] = pos | (covered << 8);
            }
        }
    }
}

// Everything that is derived from the stored arrays of a format (used by the builder and by deserialization):
// shared-memory sizing statistics, the device-only work lists and start-bit table, the decoding tables.
void finish_derived(Format& f) {
    const bool sparse = f.sparse;
    const int64_t n = f.n, m = f.m;
    const uint32_t S = f.S;
    make_decode_tables(f);
    // per-segment statistics used to size shared memory and to pick the reduction path
    const size_t U = f.seg_bit_off.size();
    f.max_unit_chunks = 1;
    f.max_sub_chunks = 1;
    for (size_t u = 0; u < U; ++u) {
        uint64_t bits = 0;
        for (int l = 0; l < 32; ++l) bits += f.sub_bits[u * 32 + l];
        const uint64_t first_chunk = f.seg_bit_off[u] >> 7;
        const uint64_t last_word = ((f.seg_bit_off[u] + bits) >> 5) + 2;
        f.max_unit_chunks = std::max<uint32_t>(f.max_unit_chunks, (uint32_t)((last_word >> 2) - first_chunk + 1));
        uint64_t at = f.seg_bit_off[u];
        for (int l = 0; l < 32; ++l) {
            const uint64_t sub_last_word = ((at + f.sub_bits[u * 32 + l]) >> 5) + 2;
            f.max_sub_chunks = std::max<uint32_t>(f.max_sub_chunks, (uint32_t)((sub_last_word >> 2) - (at >> 7) + 1));
            at += f.sub_bits[u * 32 + l];
        }
    }
    if (sparse) {
        // device-only work list: an item is one or two consecutive segments of one column
        f.item_info.clear();
        for (int64_t j = 0; j < m; ++j) {
            const uint32_t u_begin = f.seg_first[j], u_end = f.seg_first[j + 1];
            for (uint32_t u = u_begin; u < u_end; u += 2) {
                const uint32_t in_item = std::min(2u, u_end - u);
                uint32_t rec[kItemWords] = {0};
                for (uint32_t c = 0; c < in_item; ++c) {
                    // the segment's 32 sub-segment bit lengths, so that one read brings all an item needs
                    for (uint32_t l = 0; l < 32; ++l) {
                        const uint32_t bits = f.sub_bits[(size_t)(u + c) * 32 + l];
                        rec[12 + 16 * c + l / 2] |= bits << (16 * (l & 1u));
                    }
                    const uint32_t pos0 = f.cb[j] + (u + c - u_begin) * 32u * S;
                    rec[4 * c + 0] = (uint32_t)(f.seg_bit_off[u + c] & 0xffffffffu);
                    rec[4 * c + 1] = (uint32_t)(f.seg_bit_off[u + c] >> 32);
                    rec[4 * c + 2] = pos0;
                    rec[4 * c + 3] = std::min<uint32_t>(32u * S, f.cb[j + 1] - pos0);
                }
                rec[8] = (uint32_t)j;
                rec[9] = in_item | ((u_end - u_begin) <= 2 ? 0x100u : 0u);   // bit 8: the item is the whole column
                rec[10] = u;
                f.item_info.insert(f.item_info.end(), rec, rec + kItemWords);
            }
        }
        f.max_units_per_col = 0;
        f.has_empty_col = false;
        for (int64_t j = 0; j < m; ++j) {
            const uint32_t g = f.seg_first[j + 1] - f.seg_first[j];
            f.max_units_per_col = std::max(f.max_units_per_col, g);
            if (g == 0) f.has_empty_col = true;
        }
        // Row tasks of the batched tensor-core kernel.  Every lane of that kernel keeps a private copy of its
        // column's span of the stream and slice of ri for the task at hand, so the task length is the largest
        // power of two (16 .. 1024 rows) for which the fullest task of any column fits 128 bytes of such buffers.
        f.task_off.clear(); f.task_pos.clear(); f.tc_rows = 0;
        f.max_task_chunks = 1; f.max_task_ri_chunks = 1;
        if (f.nnz > 0) {
            // code word length of every stored entry (canonical code: first length whose range holds the window)
            std::vector<uint8_t> entry_len((size_t)f.nnz);
            {
                const DecodeTables& tb = f.tables;
                uint64_t bit = 0;
                for (int64_t q = 0; q < f.nnz; ++q) {
                    const uint64_t wi = bit >> 5;
                    const uint32_t sh = (uint32_t)(bit & 31);
                    const uint64_t two = ((uint64_t)f.stream[wi] << 32) | f.stream[wi + 1];
                    const uint32_t top = (uint32_t)((two << sh) >> 32);
                    uint32_t len = f.max_len;
                    for (uint32_t l = f.min_len; l <= f.max_len; ++l)
                        if ((uint64_t)top < tb.limit[l]) { len = l; break; }
                    entry_len[(size_t)q] = (uint8_t)len;
                    bit += len;
                }
            }
            const uint32_t row_bytes = f.ri_bits / 8;
            for (uint32_t T = 1024; T >= 16; T /= 2) {
                const uint64_t tasks = ((uint64_t)n + T - 1) / T;
                if ((tasks + 1) * (uint64_t)m * 12 > kTaskOffBytesMax) break;      // smaller tasks only need more
                std::vector<uint64_t> off((size_t)((tasks + 1) * (uint64_t)m), 0);
                std::vector<uint32_t> pos((size_t)((tasks + 1) * (uint64_t)m), 0);
                uint32_t max_s = 1, max_r = 1;
                uint64_t bit = 0;
                for (int64_t j = 0; j < m; ++j) {
                    uint64_t t = 0;                       // next task whose start has not been recorded yet
                    auto record = [&](uint32_t p) { off[(size_t)t * m + j] = bit; pos[(size_t)t * m + j] = p; ++t; };
                    for (uint32_t q = f.cb[j]; q < f.cb[j + 1]; ++q) {
                        const uint64_t row = f.ri_bits == 16 ? f.ri16[q] : f.ri32[q];
                        while (t <= tasks && t * T <= row) record(q);
                        bit += entry_len[q];
                    }
                    while (t <= tasks) record(f.cb[j + 1]);
                    for (uint64_t tt = 0; tt < tasks; ++tt) {
                        const uint64_t b0 = off[(size_t)tt * m + j], b1 = off[(size_t)(tt + 1) * m + j];
                        const uint64_t last_word = (b1 >> 5) + 2;
                        max_s = std::max<uint32_t>(max_s, (uint32_t)((last_word >> 2) - (b0 >> 7) + 1));
                        const uint64_t p0 = (uint64_t)pos[(size_t)tt * m + j] * row_bytes;
                        const uint64_t p1 = (uint64_t)pos[(size_t)(tt + 1) * m + j] * row_bytes;
                        max_r = std::max<uint32_t>(max_r, (uint32_t)(((p1 + 15) >> 4) - (p0 >> 4) + 1));
                    }
                }
                if (max_s + max_r <= 8 || T == 16) {
                    f.tc_rows = T; f.task_off.swap(off); f.task_pos.swap(pos);
                    f.max_task_chunks = max_s; f.max_task_ri_chunks = max_r;
                    break;
                }
            }
        }
    } else {
        f.max_units_per_col = f.G;
        const uint64_t tasks = ((uint64_t)n + S - 1) / S;
        f.task_off.clear();
        if ((tasks + 1) * (uint64_t)m * 8 <= kTaskOffBytesMax) {
            f.task_off.assign((size_t)((tasks + 1) * (uint64_t)m), 0);
            for (int64_t j = 0; j < m; ++j) {
                uint64_t t = 0;
                for (uint32_t g = 0; g < f.G; ++g) {
                    const size_t u = (size_t)j * f.G + g;
                    uint64_t at = f.seg_bit_off[u];
                    for (uint32_t l = 0; l < 32 && t < tasks; ++l, ++t) {
                        f.task_off[(size_t)t * m + j] = at;
                        at += f.sub_bits[u * 32 + l];
                    }
                    if (t == tasks) f.task_off[(size_t)tasks * m + j] = at;
                }
            }
        }
    }
}

// One matrix on its way through the builder: checked, copied column-major and pruned (Sect. III-B).
struct Layer {
    Format* f = nullptr;
    std::vector<float> col;          // pruned weights, column-major
    int64_t first = 0;               // position of its first non-null weight among those of all layers
};

static int check_params(const hac_build_params* p) {
    if (!p) return HAC_ERR_INVALID_ARG;
    if (!(p->sparsity >= 0.0 && p->sparsity < 1.0) || p->reserved != 0) return HAC_ERR_INVALID_ARG;
    if (p->quantizer > HAC_QUANT_PWS) return HAC_ERR_INVALID_ARG;
    if (p->quantizer == HAC_QUANT_KMEANS && p->k < 1) return HAC_ERR_INVALID_ARG;
    if (p->quantizer >= HAC_QUANT_UNIFORM && p->k < 2) return HAC_ERR_INVALID_ARG;
    if (p->seg_symbols > HAC_MAX_SEG_SYMBOLS) return HAC_ERR_INVALID_ARG;
    if (p->ri_bits != 0 && p->ri_bits != 16 && p->ri_bits != 32) return HAC_ERR_INVALID_ARG;
    return HAC_OK;
}

static int prepare_layer(const float* W, int64_t n, int64_t m, int64_t ldw, const hac_build_params* p, bool sparse,
                         Layer& L) {
    Format& f = *L.f;
    if (!W || n < 1 || m < 1 || ldw < m) return HAC_ERR_INVALID_ARG;
    if (n > (int64_t)1 << 31 || m > (int64_t)1 << 31 || n * m > ((int64_t)1 << 36))
        return HAC_ERR_OFFSET_OVERFLOW;
    f.sparse = sparse;
    f.n = n; f.m = m;
    f.ri_bits = sparse ? (p->ri_bits ? p->ri_bits : (n <= 65536 ? 16u : 32u)) : 0u;
    f.S = p->seg_symbols ? p->seg_symbols : (sparse ? 0u : 64u);   // sHAC default: chosen from the data below
    if (sparse && f.ri_bits == 16 && n > 65536) return HAC_ERR_INVALID_ARG;
    const int64_t total = n * m;

    // column-major copy, input checks
    std::vector<float>& col = L.col;
    col.resize(total);
    for (int64_t i = 0; i < n; ++i) {
        const float* row = W + i * ldw;
        for (int64_t j = 0; j < m; ++j) {
            float v = row[j];
            if (!std::isfinite(v)) return HAC_ERR_NONFINITE_INPUT;
            col[j * n + i] = (v == 0.0f) ? 0.0f : v;
        }
    }
    // Sect. III-B: threshold = z-th smallest magnitude, entries at or below it go
    const int64_t z = (int64_t)std::floor(p->sparsity * (double)total);
    if (z > 0) {
        std::vector<float> mag(total);
        for (int64_t t = 0; t < total; ++t) mag[t] = std::fabs(col[t]);
        std::nth_element(mag.begin(), mag.begin() + (z - 1), mag.end());
        const float tau = mag[z - 1];
        for (int64_t t = 0; t < total; ++t)
            if (std::fabs(col[t]) <= tau) col[t] = 0.0f;
    }
    // non-null weights in column-major order
    int64_t q = 0;
    for (int64_t t = 0; t < total; ++t) q += (col[t] != 0.0f);
    f.nnz = q;
    if (q >= ((int64_t)1 << 32)) return HAC_ERR_OFFSET_OVERFLOW;
    if (f.S == 0) {
        // sHAC default: two segments cover the fullest column, and the sub-segments' slices of ri
        // start an odd number of 32-bit words apart (keeps the 32 lanes on distinct shared-memory banks)
        int64_t fullest = 0;
        for (int64_t j = 0; j < m; ++j) {
            int64_t c = 0;
            const float* cj = col.data() + j * n;
            for (int64_t i = 0; i < n; ++i) c += (cj[i] != 0.0f);
            fullest = std::max(fullest, c);
        }
        uint32_t S = (uint32_t)std::min<int64_t>(256, std::max<int64_t>(4, (fullest + 63) / 64));
        if (f.ri_bits == 16) { while (S % 4 != 2) ++S; } else { S |= 1u; }
        f.S = S;
    }
    return HAC_OK;
}

// Sect. IV-B / IV-C: emit the code words of one matrix column by column with the given code, recording the
// offset index on the way.  level_of: the shared level of each of its non-null weights, in column-major order.
static int emit_layer(Layer& L, const uint32_t* level_of, const std::vector<uint32_t>& level_symbol, uint32_t zero_symbol,
                      const std::vector<float>& values, const std::vector<uint8_t>& code_len, const std::vector<uint32_t>& codes) {
    Format& f = *L.f;
    const std::vector<float>& col = L.col;
    const bool sparse = f.sparse;
    const int64_t n = f.n, m = f.m, total = n * m, q = f.nnz;
    const uint32_t k_eff = (uint32_t)values.size();
    f.codebook = values;
    f.code_len = code_len;
    f.codes = codes;
    f.counts.assign(k_eff, 0);
    f.max_len = 0; f.min_len = k_eff ? 255 : 0;
    for (uint8_t l : f.code_len) { f.max_len = std::max<uint32_t>(f.max_len, l); f.min_len = std::min<uint32_t>(f.min_len, l); }
    if ((uint64_t)f.S * f.max_len > 65535u) return HAC_ERR_OFFSET_OVERFLOW;   // sub_bits is 16 bit

    const uint32_t S = f.S;
    BitWriter bw(f.stream);
    f.symbols = sparse ? q : total;
    if (sparse) {
        f.cb.assign(m + 1, 0);
        f.seg_first.assign(m + 1, 0);
        if (f.ri_bits == 16) f.ri16.reserve(q); else f.ri32.reserve(q);
    } else {
        const uint32_t T = (uint32_t)((n + S - 1) / S);
        f.G = (T + 31) / 32;
        if ((uint64_t)f.G * (uint64_t)m >= ((uint64_t)1 << 31)) return HAC_ERR_OFFSET_OVERFLOW;
    }
    int64_t w = 0;   // running index into the non-null weights
    for (int64_t j = 0; j < m; ++j) {
        const float* c = col.data() + j * n;
        uint32_t in_sub = 0, subs_in_col = 0;
        int64_t sub_start_bit = bw.total;
        auto open_segment_if_needed = [&]() {
            if (in_sub == 0 && (subs_in_col % 32) == 0) {
                f.seg_bit_off.push_back((uint64_t)bw.total);
                f.sub_bits.resize(f.sub_bits.size() + 32, 0);
                if (sparse) f.seg_col.push_back((uint32_t)j);
            }
            if (in_sub == 0) sub_start_bit = bw.total;
        };
        auto close_sub = [&]() {
            f.sub_bits[f.sub_bits.size() - 32 + (subs_in_col % 32)] = (uint16_t)(bw.total - sub_start_bit);
            ++subs_in_col;
            in_sub = 0;
        };
        for (int64_t i = 0; i < n; ++i) {
            const bool stored = (c[i] != 0.0f);
            uint32_t s;
            if (stored) s = level_symbol[level_of[w++]];
            else if (sparse) continue;
            else s = zero_symbol;
            open_segment_if_needed();
            bw.put(f.codes[s], f.code_len[s]);
            f.counts[s]++;
            if (sparse) { if (f.ri_bits == 16) f.ri16.push_back((uint16_t)i); else f.ri32.push_back((uint32_t)i); }
            if (++in_sub == S) close_sub();
        }
        if (in_sub > 0) close_sub();
        if (sparse) {
            f.cb[j + 1] = (uint32_t)w;
            f.seg_first[j + 1] = (uint32_t)f.seg_bit_off.size();
        }
    }
    bw.finish();
    f.stream_bits = bw.total;
    f.stream_words = (int64_t)f.stream.size();
    const int64_t padded = ((f.stream_words + 3) / 4) * 4 + kStreamSlackWords;
    f.pad_words = padded - f.stream_words;
    f.stream.resize(padded, 0u);

    finish_derived(f);
    return HAC_OK;
}

// Weight sharing over the non-null weights of all the layers at once (one layer: Sect. III-C; several: the unified
// quantization of Sect. V-D, one k and one dictionary for all of them), one Huffman code on the symbol counts of all the
// streams together, then every layer emitted with that code.  A layer keeps the whole shared codebook and code and its
// own symbol counts.
int build_layers(std::vector<Layer>& layers, const hac_build_params* p) {
    std::vector<double> data;
    int64_t q_all = 0, nulls_in_hac = 0;
    for (Layer& L : layers) {
        L.first = q_all;
        q_all += L.f->nnz;
        if (!L.f->sparse) nulls_in_hac += L.f->n * L.f->m - L.f->nnz;
    }
    data.reserve(q_all);
    for (const Layer& L : layers)
        for (float v : L.col)
            if (v != 0.0f) data.push_back((double)v);

    Shared sh;
    if (q_all > 0) {
        int rc = HAC_OK;
        if (p->quantizer == HAC_QUANT_KMEANS) rc = share_kmeans(data, p->k, p->kmeans_iters, p->seed, sh);
        else if (p->quantizer == HAC_QUANT_UNIFORM) rc = share_uniform(data, p->k, sh);
        else if (p->quantizer == HAC_QUANT_GRID) rc = share_grid(data, p->k, sh);
        else if (p->quantizer == HAC_QUANT_PWS) rc = share_pws(data, p->k, p->seed, sh);
        else rc = share_none(data, sh);
        if (rc != HAC_OK) return rc;
    }
    std::vector<double>().swap(data);
    for (float& v : sh.level_value) if (v == 0.0f) v = 0.0f;           // -0.0 -> +0.0

    // alphabet: occupied levels (plus zero when a HAC layer has a null entry), merged by value.  A stored entry of an
    // sHAC layer is counted like any other occurrence of its value.
    const size_t nlev = sh.level_value.size();
    std::vector<int64_t> level_count(nlev, 0);
    for (int64_t t = 0; t < q_all; ++t) level_count[sh.level_of[t]]++;
    std::vector<float> values;
    for (size_t l = 0; l < nlev; ++l) if (level_count[l] > 0) values.push_back(sh.level_value[l]);
    if (nulls_in_hac > 0) values.push_back(0.0f);
    std::sort(values.begin(), values.end());
    values.erase(std::unique(values.begin(), values.end()), values.end());
    if (values.size() > HAC_MAX_SYMBOLS) return HAC_ERR_K_TOO_LARGE;
    const uint32_t k_eff = (uint32_t)values.size();
    std::vector<uint32_t> level_symbol(nlev, 0);
    for (size_t l = 0; l < nlev; ++l)
        level_symbol[l] = (uint32_t)(std::lower_bound(values.begin(), values.end(), sh.level_value[l]) -
                                     values.begin());
    uint32_t zero_symbol = 0;
    if (nulls_in_hac > 0)
        zero_symbol = (uint32_t)(std::lower_bound(values.begin(), values.end(), 0.0f) - values.begin());
    std::vector<int64_t> counts(k_eff, 0);
    for (size_t l = 0; l < nlev; ++l) if (level_count[l] > 0) counts[level_symbol[l]] += level_count[l];
    if (nulls_in_hac > 0) counts[zero_symbol] += nulls_in_hac;

    std::vector<uint8_t> code_len;
    std::vector<uint32_t> codes;
    int rc = huffman_code_lengths(counts, code_len);
    if (rc != HAC_OK) return rc;
    canonical_assign(code_len, codes);
    for (Layer& L : layers) {
        rc = emit_layer(L, sh.level_of.data() + L.first, level_symbol, zero_symbol, values, code_len, codes);
        if (rc != HAC_OK) return rc;
        std::vector<float>().swap(L.col);
    }
    return HAC_OK;
}

int build_impl(const float* W, int64_t n, int64_t m, int64_t ldw, const hac_build_params* p,
                      bool sparse, Format& f) {
    if (int rc = check_params(p)) return rc;
    std::vector<Layer> layers(1);
    layers[0].f = &f;
    if (int rc = prepare_layer(W, n, m, ldw, p, sparse, layers[0])) return rc;
    return build_layers(layers, p);
}

// Host decoder (canonical decoding by lengths, one symbol at a time); used by *_decode_host.
int decode_on_host(const Format& f, float* Wq, int64_t ldq) {
    if (!Wq || ldq < f.m) return HAC_ERR_INVALID_ARG;
    for (int64_t i = 0; i < f.n; ++i) std::fill(Wq + i * ldq, Wq + i * ldq + f.m, 0.0f);
    const DecodeTables& t = f.tables;
    uint64_t bit = 0;
    auto next_value = [&](float& v) -> bool {
        uint64_t wi = bit >> 5;
        uint32_t sh = (uint32_t)(bit & 31);
        if ((int64_t)wi + 1 >= (int64_t)f.stream.size()) return false;
        uint64_t two = ((uint64_t)f.stream[wi] << 32) | f.stream[wi + 1];
        uint32_t top = (uint32_t)((two << sh) >> 32);
        for (uint32_t l = f.min_len; l <= f.max_len; ++l) {
            if ((uint64_t)top < t.limit[l]) {
                uint32_t r = t.rank_base[l] + ((top - t.first_left[l]) >> (32 - l));
                if (r >= t.rank_value.size()) return false;
                v = t.rank_value[r];
                bit += l;
                return true;
            }
        }
        return false;
    };
    if (!f.sparse) {
        for (int64_t j = 0; j < f.m; ++j)
            for (int64_t i = 0; i < f.n; ++i) {
                float v;
                if (!next_value(v)) return HAC_ERR_CORRUPT;
                Wq[i * ldq + j] = v;
            }
    } else {
        for (int64_t j = 0; j < f.m; ++j)
            for (uint32_t p = f.cb[j]; p < f.cb[j + 1]; ++p) {
                float v;
                if (!next_value(v)) return HAC_ERR_CORRUPT;
                const int64_t i = f.ri_bits == 16 ? (int64_t)f.ri16[p] : (int64_t)f.ri32[p];
                Wq[i * ldq + j] = v;
            }
    }
    return (int64_t)bit == f.stream_bits ? HAC_OK : HAC_ERR_CORRUPT;
}

void fill_size_report(const Format& f, hac_size_report* r) {
    std::memset(r, 0, sizeof(*r));
    r->n = f.n; r->m = f.m; r->nnz = f.nnz; r->symbols = f.symbols;
    r->stream_bits = f.stream_bits;
    r->stream_words = f.stream_words;
    r->stream_bytes = 4 * f.stream_words;
    r->pad_bytes = 4 * f.pad_words;
    r->codebook_bytes = 4 * (int64_t)f.codebook.size();
    r->code_len_bytes = (int64_t)f.code_len.size();
    r->ri_bytes = f.sparse ? f.nnz * (int64_t)f.ri_bits / 8 : 0;
    r->cb_bytes = f.sparse ? 4 * (f.m + 1) : 0;
    r->offset_index_bytes = (int64_t)(f.seg_bit_off.size() * 8 + f.sub_bits.size() * 2 +
                                      f.seg_first.size() * 4 + f.seg_col.size() * 4);
    r->total_bytes = r->stream_bytes + r->pad_bytes + r->codebook_bytes + r->code_len_bytes +
                     r->ri_bytes + r->cb_bytes + r->offset_index_bytes;
    const int64_t k = (int64_t)f.codebook.size();
    const double logk = k > 0 ? std::log2((double)k) : 0.0;
    if (!f.sparse) {
        r->paper_bits = 32 * f.stream_words + 6 * k * 32;
        r->bound_bits = (double)f.n * (double)f.m * (1.0 + logk) + 6.0 * k * 32;
    } else {
        r->paper_bits = 32 * f.stream_words + 6 * k * 32 + 32 * (f.nnz + f.m + 1);
        r->bound_bits = (double)f.nnz * (1.0 + logk) + 32.0 * (6.0 * k + (double)f.nnz + f.m + 1);
    }
    double H = 0.0;
    for (int64_t c : f.counts)
        if (c > 0) { double pr = (double)c / (double)f.symbols; H -= pr * std::log2(pr); }
    r->entropy = H;
    r->avg_code_len = f.symbols ? (double)f.stream_bits / (double)f.symbols : 0.0;
    r->k_eff = (uint32_t)k;
    r->max_code_len = f.max_len; r->min_code_len = f.min_len;
    r->seg_symbols = f.S; r->ri_bits = f.ri_bits;
    r->units = (uint32_t)f.seg_bit_off.size();
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

ImageLayout image_layout(const Format& f) {
    ImageLayout L{};
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align256(o + std::max<size_t>(bytes, 16)); return at; };
    L.stream = take(f.stream.size() * 4);
    L.lut = take(f.tables.lut.size() * 2);
    L.l1 = take(f.tables.l1.size() * 4);
    L.sub = take(f.tables.sub.size() * 4);
    L.l1_runs = take(f.tables.l1_runs.size() * 4);
    L.xt = take(f.tables.xt.size() * 4);
    L.rank_value = take(f.tables.rank_value.size() * 4);
    L.limit = take(sizeof(f.tables.limit));
    L.first_left = take(sizeof(f.tables.first_left));
    L.rank_base = take(sizeof(f.tables.rank_base));
    L.seg_bit_off = take(f.seg_bit_off.size() * 8);
    L.sub_bits = take(f.sub_bits.size() * 2);
    L.seg_col = take(f.seg_col.size() * 4);
    L.seg_first = take(f.seg_first.size() * 4);
    L.ri = take(f.ri_bits == 16 ? f.ri16.size() * 2 + 16 : f.ri32.size() * 4 + 16);
    L.cb = take(f.cb.size() * 4);
    L.unit_info = take(f.item_info.size() * 4);
    L.task_off = take(f.task_off.size() * 8);
    L.task_pos = take(f.task_pos.size() * 4);
    L.total = o;
    return L;
}


// ------------------------------------------------------------------------------------------------
// Flat little-endian image of a built format (what has to be stored to use it later; everything
// derived is rebuilt on load).  Layout: 16 header words of 64 bits, then the arrays in the order of
// write_arrays(), each padded to 8 bytes, then a 64-bit FNV-1a checksum of all bytes before it.
// ------------------------------------------------------------------------------------------------
static const uint64_t kBlobMagic = 0x3130424341480aefull;      // "\xef\nHACB01"
static const uint64_t kBlobVersion = 1;

static uint64_t fnv1a(const unsigned char* p, size_t n) {
    uint64_t h = 0xcbf29ce484222325ull;
    for (size_t i = 0; i < n; ++i) { h ^= p[i]; h *= 0x100000001b3ull; }
    return h;
}
static size_t pad8(size_t x) { return (x + 7) & ~(size_t)7; }

struct BlobSizes { size_t codebook, code_len, counts, stream, seg_bit_off, sub_bits, seg_first, seg_col, ri, cb, total; };
static BlobSizes blob_sizes(bool sparse, uint64_t k, uint64_t stream_words_padded, uint64_t units, uint64_t m, uint64_t nnz,
                            uint32_t ri_bits) {
    BlobSizes b{};
    b.codebook = pad8(k * 4); b.code_len = pad8(k); b.counts = k * 8; b.stream = pad8(stream_words_padded * 4);
    b.seg_bit_off = units * 8; b.sub_bits = pad8(units * 64);
    b.seg_first = sparse ? pad8((m + 1) * 4) : 0; b.seg_col = sparse ? pad8(units * 4) : 0;
    b.ri = sparse ? pad8(nnz * (ri_bits / 8)) : 0; b.cb = sparse ? pad8((m + 1) * 4) : 0;
    b.total = 16 * 8 + b.codebook + b.code_len + b.counts + b.stream + b.seg_bit_off + b.sub_bits + b.seg_first + b.seg_col +
              b.ri + b.cb + 8;
    return b;
}

static size_t serialized_bytes(const Format& f) {
    return blob_sizes(f.sparse, f.codebook.size(), f.stream.size(), f.seg_bit_off.size(), (uint64_t)f.m, (uint64_t)f.nnz,
                      f.ri_bits ? f.ri_bits : 32).total;
}

static int serialize(const Format& f, void* buf, size_t bytes) {
    if (!buf) return HAC_ERR_INVALID_ARG;
    const size_t need = serialized_bytes(f);
    if (bytes < need) return HAC_ERR_BUFFER_TOO_SMALL;
    unsigned char* p = static_cast<unsigned char*>(buf);
    std::memset(p, 0, need);
    const uint64_t hdr[16] = {kBlobMagic, kBlobVersion, f.sparse ? 1u : 0u, (uint64_t)f.n, (uint64_t)f.m, (uint64_t)f.nnz,
                              (uint64_t)f.symbols, f.S, f.G, f.ri_bits, (uint64_t)f.codebook.size(), (uint64_t)f.stream_bits,
                              (uint64_t)f.stream_words, (uint64_t)f.pad_words, (uint64_t)f.seg_bit_off.size(), 0};
    std::memcpy(p, hdr, sizeof(hdr));
    size_t o = sizeof(hdr);
    auto put = [&](const void* src, size_t n) { if (n) std::memcpy(p + o, src, n); o += pad8(n); };
    put(f.codebook.data(), f.codebook.size() * 4);
    put(f.code_len.data(), f.code_len.size());
    put(f.counts.data(), f.counts.size() * 8);
    put(f.stream.data(), f.stream.size() * 4);
    put(f.seg_bit_off.data(), f.seg_bit_off.size() * 8);
    put(f.sub_bits.data(), f.sub_bits.size() * 2);
    if (f.sparse) {
        put(f.seg_first.data(), f.seg_first.size() * 4);
        put(f.seg_col.data(), f.seg_col.size() * 4);
        if (f.ri_bits == 16) put(f.ri16.data(), f.ri16.size() * 2); else put(f.ri32.data(), f.ri32.size() * 4);
        put(f.cb.data(), f.cb.size() * 4);
    }
    const uint64_t sum = fnv1a(p, o);
    std::memcpy(p + o, &sum, 8);
    return HAC_OK;
}

// Rebuilds a format from its image.  Everything is checked before it is used: sizes against the header,
// the checksum, the code (lengths between 1 and 32 that satisfy the Kraft equality, values strictly
// ascending, counts that add up to the number of code words and to the length of the stream), the offset
// index (segments in stream order, sub-segment lengths that tile the stream) and, for sHAC, cb, ri and
// the segment lists.  Anything else is HAC_ERR_CORRUPT.
static int deserialize(const void* buf, size_t bytes, bool want_sparse, Format& f) {
    if (!buf) return HAC_ERR_INVALID_ARG;
    const unsigned char* p = static_cast<const unsigned char*>(buf);
    if (bytes < 16 * 8 + 8) return HAC_ERR_CORRUPT;
    uint64_t hdr[16];
    std::memcpy(hdr, p, sizeof(hdr));
    if (hdr[0] != kBlobMagic || hdr[1] != kBlobVersion || hdr[2] > 1 || hdr[15] != 0) return HAC_ERR_CORRUPT;
    const bool sparse = hdr[2] == 1;
    if (sparse != want_sparse) return HAC_ERR_INVALID_ARG;
    const uint64_t n = hdr[3], m = hdr[4], nnz = hdr[5], symbols = hdr[6], S = hdr[7], G = hdr[8], ri_bits = hdr[9], k = hdr[10],
                   stream_bits = hdr[11], stream_words = hdr[12], pad_words = hdr[13], units = hdr[14];
    if (n < 1 || m < 1 || n > ((uint64_t)1 << 31) || m > ((uint64_t)1 << 31) || n * m > ((uint64_t)1 << 36)) return HAC_ERR_CORRUPT;
    if (S < 1 || S > HAC_MAX_SEG_SYMBOLS || k > HAC_MAX_SYMBOLS || nnz > n * m) return HAC_ERR_CORRUPT;
    if (symbols != (sparse ? nnz : n * m) || (symbols > 0 && k == 0)) return HAC_ERR_CORRUPT;
    if (sparse ? (ri_bits != 16 && ri_bits != 32) || (ri_bits == 16 && n > 65536) || G != 0 : ri_bits != 0) return HAC_ERR_CORRUPT;
    if (stream_words != (stream_bits + 31) / 32 || pad_words != ((stream_words + 3) / 4) * 4 + kStreamSlackWords - stream_words)
        return HAC_ERR_CORRUPT;
    if (!sparse && (G != ((n + S - 1) / S + 31) / 32 || units != G * m)) return HAC_ERR_CORRUPT;
    if (units > ((uint64_t)1 << 31)) return HAC_ERR_CORRUPT;
    const BlobSizes bs = blob_sizes(sparse, k, stream_words + pad_words, units, m, nnz, (uint32_t)(ri_bits ? ri_bits : 32));
    if (bs.total != bytes) return HAC_ERR_CORRUPT;
    uint64_t sum;
    std::memcpy(&sum, p + bytes - 8, 8);
    if (sum != fnv1a(p, bytes - 8)) return HAC_ERR_CORRUPT;

    f = Format();
    f.sparse = sparse; f.n = (int64_t)n; f.m = (int64_t)m; f.nnz = (int64_t)nnz; f.symbols = (int64_t)symbols;
    f.S = (uint32_t)S; f.G = (uint32_t)G; f.ri_bits = (uint32_t)ri_bits;
    f.stream_bits = (int64_t)stream_bits; f.stream_words = (int64_t)stream_words; f.pad_words = (int64_t)pad_words;
    size_t o = sizeof(hdr);
    auto get = [&](void* dst, size_t nbytes) { if (nbytes) std::memcpy(dst, p + o, nbytes); o += pad8(nbytes); };
    f.codebook.resize(k); get(f.codebook.data(), k * 4);
    f.code_len.resize(k); get(f.code_len.data(), k);
    f.counts.resize(k); get(f.counts.data(), k * 8);
    f.stream.resize(stream_words + pad_words); get(f.stream.data(), f.stream.size() * 4);
    f.seg_bit_off.resize(units); get(f.seg_bit_off.data(), units * 8);
    f.sub_bits.resize(units * 32); get(f.sub_bits.data(), units * 64);
    if (sparse) {
        f.seg_first.resize(m + 1); get(f.seg_first.data(), (m + 1) * 4);
        f.seg_col.resize(units); get(f.seg_col.data(), units * 4);
        if (ri_bits == 16) { f.ri16.resize(nnz); get(f.ri16.data(), nnz * 2); }
        else { f.ri32.resize(nnz); get(f.ri32.data(), nnz * 4); }
        f.cb.resize(m + 1); get(f.cb.data(), (m + 1) * 4);
    }
    // the code
    f.max_len = 0; f.min_len = k ? 255 : 0;
    long double kraft = 0;
    uint64_t total_count = 0, total_bits = 0;
    for (uint64_t s = 0; s < k; ++s) {
        const uint32_t l = f.code_len[s];
        if (l < 1 || l > (uint32_t)kMaxCodeLen || f.counts[s] < 0) return HAC_ERR_CORRUPT;   // 0: a symbol of a shared code that this matrix lacks
        if (!std::isfinite(f.codebook[s]) || (s > 0 && !(f.codebook[s] > f.codebook[s - 1]))) return HAC_ERR_CORRUPT;
        kraft += std::ldexp((long double)1, -(int)l);
        total_count += (uint64_t)f.counts[s]; total_bits += (uint64_t)f.counts[s] * l;
        f.max_len = std::max(f.max_len, l); f.min_len = std::min(f.min_len, l);
    }
    if (k == 1 ? f.code_len[0] != 1 : (k >= 2 && kraft != 1)) return HAC_ERR_CORRUPT;
    if (total_count != symbols || total_bits != stream_bits || S * f.max_len > 65535u) return HAC_ERR_CORRUPT;
    for (uint64_t w = stream_words; w < stream_words + pad_words; ++w) if (f.stream[w] != 0) return HAC_ERR_CORRUPT;
    if (stream_bits & 31u) { if (f.stream[stream_words - 1] & ((1u << (32 - (stream_bits & 31u))) - 1u)) return HAC_ERR_CORRUPT; }
    canonical_assign(f.code_len, f.codes);
    // the offset index: segments tile the stream in order
    uint64_t at = 0;
    for (uint64_t u = 0; u < units; ++u) {
        if (f.seg_bit_off[u] != at) return HAC_ERR_CORRUPT;
        for (int l = 0; l < 32; ++l) at += f.sub_bits[u * 32 + l];
    }
    if (at != stream_bits) return HAC_ERR_CORRUPT;
    if (sparse) {
        if (f.cb[0] != 0 || f.cb[m] != nnz || f.seg_first[0] != 0 || f.seg_first[m] != units) return HAC_ERR_CORRUPT;
        for (uint64_t j = 0; j < m; ++j) {
            if (f.cb[j + 1] < f.cb[j] || f.seg_first[j + 1] < f.seg_first[j]) return HAC_ERR_CORRUPT;
            const uint64_t entries = f.cb[j + 1] - f.cb[j];
            if (f.seg_first[j + 1] - f.seg_first[j] != (entries + 32 * S - 1) / (32 * S)) return HAC_ERR_CORRUPT;
            for (uint32_t u = f.seg_first[j]; u < f.seg_first[j + 1]; ++u) if (f.seg_col[u] != j) return HAC_ERR_CORRUPT;
            for (uint64_t q = f.cb[j]; q < f.cb[j + 1]; ++q) {
                const uint64_t r = ri_bits == 16 ? f.ri16[q] : f.ri32[q];
                if (r >= n || (q > f.cb[j] && r <= (ri_bits == 16 ? (uint64_t)f.ri16[q - 1] : (uint64_t)f.ri32[q - 1]))) return HAC_ERR_CORRUPT;
            }
        }
    }
    finish_derived(f);
    return HAC_OK;
}

}  // namespace hacb200

using hacb200::Format;

// What the first-level decoding table of the kernels holds for a 32-bit window (test support).
static int table_lookup_host(const Format& f, uint32_t window, float* value, uint32_t* length, int* kind,
                             int* never_unresolved) {
    if (!value || !length || !kind || !never_unresolved) return HAC_ERR_INVALID_ARG;
    const hacb200::DecodeTables& t = f.tables;
    uint32_t v = 0, meta = 0;
    if (t.use_xt) {
        const uint32_t low = f.max_len < 32u ? ((1u << (32u - f.max_len)) - 1u) | 1u : 1u;
        const uint32_t idx = hacb200::xt_index(~(~window | low), t.xt_mant);     // the index the kernels form from ~window | low
        v = t.xt[2 * (size_t)idx]; meta = t.xt[2 * (size_t)idx + 1];
        *kind = 1;
        *never_unresolved = t.xt_unresolved == 0.0;
    } else {
        if (t.l1.empty()) return HAC_ERR_INVALID_ARG;
        const uint32_t idx = t.l1_bits >= 32 ? window : window >> (32 - t.l1_bits);
        v = t.l1[2 * (size_t)idx]; meta = t.l1[2 * (size_t)idx + 1];
        *kind = 0;
        *never_unresolved = f.max_len <= (uint32_t)t.l1_bits;
    }
    if (meta & 0x80000000u) { *length = 0; *value = 0.0f; }
    else { *length = meta; std::memcpy(value, &v, 4); }
    return HAC_OK;
}

extern "C" {

int hac_serialize_bytes(const hac_format* f, size_t* out) {
    if (!f || !out) return HAC_ERR_INVALID_ARG;
    *out = hacb200::serialized_bytes(f->f);
    return HAC_OK;
}
int shac_serialize_bytes(const shac_format* f, size_t* out) {
    if (!f || !out) return HAC_ERR_INVALID_ARG;
    *out = hacb200::serialized_bytes(f->f);
    return HAC_OK;
}
int hac_serialize(const hac_format* f, void* buf, size_t bytes) { return f ? hacb200::serialize(f->f, buf, bytes) : HAC_ERR_INVALID_ARG; }
int shac_serialize(const shac_format* f, void* buf, size_t bytes) { return f ? hacb200::serialize(f->f, buf, bytes) : HAC_ERR_INVALID_ARG; }
int hac_deserialize(const void* buf, size_t bytes, hac_format** out) {
    if (!out) return HAC_ERR_INVALID_ARG;
    *out = nullptr;
    hac_format* h = new (std::nothrow) hac_format();
    if (!h) return HAC_ERR_ALLOC;
    int rc;
    try { rc = hacb200::deserialize(buf, bytes, false, h->f); }
    catch (const std::bad_alloc&) { rc = HAC_ERR_ALLOC; }
    if (rc != HAC_OK) { delete h; return rc; }
    *out = h;
    return HAC_OK;
}
int shac_deserialize(const void* buf, size_t bytes, shac_format** out) {
    if (!out) return HAC_ERR_INVALID_ARG;
    *out = nullptr;
    shac_format* h = new (std::nothrow) shac_format();
    if (!h) return HAC_ERR_ALLOC;
    int rc;
    try { rc = hacb200::deserialize(buf, bytes, true, h->f); }
    catch (const std::bad_alloc&) { rc = HAC_ERR_ALLOC; }
    if (rc != HAC_OK) { delete h; return rc; }
    *out = h;
    return HAC_OK;
}

int hac_debug_table_lookup(const hac_format* f, uint32_t window, float* value, uint32_t* length, int* kind,
                           int* never_unresolved) {
    return f ? table_lookup_host(f->f, window, value, length, kind, never_unresolved) : HAC_ERR_INVALID_ARG;
}
int shac_debug_table_lookup(const shac_format* f, uint32_t window, float* value, uint32_t* length, int* kind,
                            int* never_unresolved) {
    return f ? table_lookup_host(f->f, window, value, length, kind, never_unresolved) : HAC_ERR_INVALID_ARG;
}

int hac_build(const float* W, int64_t n, int64_t m, int64_t ldw, const hac_build_params* params,
              hac_format** out) {
    if (!out) return HAC_ERR_INVALID_ARG;
    *out = nullptr;
    hac_format* h = new (std::nothrow) hac_format();
    if (!h) return HAC_ERR_ALLOC;
    int rc;
    try { rc = hacb200::build_impl(W, n, m, ldw, params, false, h->f); }
    catch (const std::bad_alloc&) { rc = HAC_ERR_ALLOC; }
    if (rc != HAC_OK) { delete h; return rc; }
    *out = h;
    return HAC_OK;
}

int shac_build(const float* W, int64_t n, int64_t m, int64_t ldw, const hac_build_params* params,
               shac_format** out) {
    if (!out) return HAC_ERR_INVALID_ARG;
    *out = nullptr;
    shac_format* h = new (std::nothrow) shac_format();
    if (!h) return HAC_ERR_ALLOC;
    int rc;
    try { rc = hacb200::build_impl(W, n, m, ldw, params, true, h->f); }
    catch (const std::bad_alloc&) { rc = HAC_ERR_ALLOC; }
    if (rc != HAC_OK) { delete h; return rc; }
    *out = h;
    return HAC_OK;
}

int hac_build_unified(const hac_unified_layer* layers, int n_layers, const hac_build_params* params, void** out) {
    if (!layers || !out || n_layers < 1 || n_layers > HAC_MAX_UNIFIED_LAYERS) return HAC_ERR_INVALID_ARG;
    for (int i = 0; i < n_layers; ++i) out[i] = nullptr;
    if (int rc = hacb200::check_params(params)) return rc;
    // hac_format and shac_format hold the same thing; which one a layer's handle is follows its `sparse` field
    std::vector<hac_format*> hs;
    std::vector<shac_format*> ss;
    auto drop = [&]() { for (auto* h : hs) delete h; for (auto* h : ss) delete h; for (int i = 0; i < n_layers; ++i) out[i] = nullptr; };
    int rc = HAC_OK;
    try {
        std::vector<hacb200::Layer> ls((size_t)n_layers);
        for (int i = 0; i < n_layers && rc == HAC_OK; ++i) {
            if (layers[i].sparse != 0 && layers[i].sparse != 1) { rc = HAC_ERR_INVALID_ARG; break; }
            if (layers[i].sparse) { ss.push_back(new shac_format()); ls[i].f = &ss.back()->f; out[i] = ss.back(); }
            else { hs.push_back(new hac_format()); ls[i].f = &hs.back()->f; out[i] = hs.back(); }
            rc = hacb200::prepare_layer(layers[i].W, layers[i].n, layers[i].m, layers[i].ldw, params, layers[i].sparse != 0, ls[i]);
        }
        if (rc == HAC_OK) rc = hacb200::build_layers(ls, params);
    } catch (const std::bad_alloc&) { rc = HAC_ERR_ALLOC; }
    if (rc != HAC_OK) drop();
    return rc;
}

int hac_sizes(const hac_format* f, hac_size_report* out) {
    if (!f || !out) return HAC_ERR_INVALID_ARG;
    hacb200::fill_size_report(f->f, out);
    return HAC_OK;
}
int shac_sizes(const shac_format* f, hac_size_report* out) {
    if (!f || !out) return HAC_ERR_INVALID_ARG;
    hacb200::fill_size_report(f->f, out);
    return HAC_OK;
}

static void fill_view(const Format& f, hac_host_view* v) {
    v->n = f.n; v->m = f.m;
    v->k_eff = (uint32_t)f.codebook.size();
    v->seg_symbols = f.S;
    v->codebook = f.codebook.data();
    v->code_len = f.code_len.data();
    v->codes = f.codes.data();
    v->counts = f.counts.data();
    v->stream = f.stream.data();
    v->stream_bits = f.stream_bits;
    v->stream_words = f.stream_words;
    v->stream_pad_words = f.pad_words;
    v->units = (uint32_t)f.seg_bit_off.size();
    v->segs_per_col = f.sparse ? 0 : f.G;
    v->seg_bit_off = f.seg_bit_off.data();
    v->sub_bits = f.sub_bits.data();
}

int hac_export(const hac_format* f, hac_host_view* out) {
    if (!f || !out) return HAC_ERR_INVALID_ARG;
    fill_view(f->f, out);
    return HAC_OK;
}
int shac_export(const shac_format* f, shac_host_view* out) {
    if (!f || !out) return HAC_ERR_INVALID_ARG;
    fill_view(f->f, &out->base);
    out->nnz = f->f.nnz;
    out->ri_bits = f->f.ri_bits;
    out->ri = f->f.ri_bits == 16 ? (const void*)f->f.ri16.data() : (const void*)f->f.ri32.data();
    out->cb = f->f.cb.data();
    out->seg_first = f->f.seg_first.data();
    out->seg_col = f->f.seg_col.data();
    return HAC_OK;
}

int hac_decode_host(const hac_format* f, float* Wq, int64_t ldq) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return hacb200::decode_on_host(f->f, Wq, ldq);
}
int shac_decode_host(const shac_format* f, float* Wq, int64_t ldq) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return hacb200::decode_on_host(f->f, Wq, ldq);
}

const char* hac_status_string(int status) {
    switch (status) {
        case HAC_OK: return "ok";
        case HAC_ERR_INVALID_ARG: return "invalid argument";
        case HAC_ERR_ALLOC: return "host allocation failed";
        case HAC_ERR_NONFINITE_INPUT: return "W holds NaN or Inf";
        case HAC_ERR_K_TOO_LARGE: return "too many distinct values";
        case HAC_ERR_CODE_TOO_LONG: return "Huffman code word longer than 32 bits";
        case HAC_ERR_OFFSET_OVERFLOW: return "size or offset overflow";
        case HAC_ERR_NOT_UPLOADED: return "format not uploaded to the device";
        case HAC_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case HAC_ERR_CUDA: return "CUDA error";
        case HAC_ERR_CORRUPT: return "corrupt data";
        default: return "unknown status";
    }
}

}  // extern "C"
