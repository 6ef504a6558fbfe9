// CPU oracle for the DISC + PPV per-step hot path.
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct
// statement of what the hot path computes.  It shares no code, header, table or
// constant generator with the CUDA library, and nothing in the product path may
// call it.  It is used by the tests, by the smoke check and by the benchmark's
// CPU-baseline leg.
//
// What it follows (paper: "Efficient and Asymptotically Unbiased Constrained
// Decoding for Large Language Models"):
//   * the valid set  A_{x,S} = { v : exists s in S with x+[v] a prefix of s }
//     (Section 2.1) is read off an explicit prefix tree whose node for path x
//     has child v iff v is in A_{x,S} (Section 2.1, "Prefix-tree");
//   * the sorted array of Algorithm 2, line 1 is the list of members in the
//     order a depth-first walk visits them when children are taken in
//     ascending token id (vocabulary order = integer order, Section 2.1
//     footnote; left-to-right comparison, Section 3.2 "Array Preparation");
//   * one decoding step is Algorithm 1, lines 5-8: mask, sample from
//     P.mask/|P.mask|_1, multiply the importance score by |P.mask|_1
//     (kept as a sum of logs; closed form in Appendix A, x(a) = prod_i
//     P_L(A_{a<i,S} | a<i));
//   * the final draw is Algorithm 1, line 22: pick candidate k with
//     probability x_k / sum_j x_j;
//   * the accept test is Algorithm 1, line 16: accept when x > eps ~ U[0,1].
//
// Readings where the paper is silent (same list as the design notes):
//   * S must be prefix-free (fixed length, or every member closed by an EOS
//     that is an ordinary token); then "a in S" is "the node is a leaf".
//   * "sample a token from the distribution" (Algorithm 1, line 7) fixes no
//     mechanism.  Two exact samplers are stated here:
//       - oracle_step_plain: the textbook inverse CDF over the allowed tokens in
//         ascending id with one uniform per (row, step).  It knows nothing of
//         how any kernel is organised and is the plain statement of line 7;
//       - oracle_step: two stages - Gumbel-max over groups of 8 consecutive
//         token ids (group score = log of the group's allowed mass + Gumbel
//         noise, one Philox4x32-10 uniform per (row, step, group), ties to the
//         lowest group), then an inverse-CDF draw inside the winning group.
//         The group size (8 ids = one 16-byte vector of bf16 logits) and the
//         counter layout of the group noise were taken from the CUDA kernel's
//         vector width and slot geometry, so that the two sides can be
//         compared token by token; the law it draws from is the same.
//     Both are pinned to the exact masked softmax (chi-square) on layouts that
//     stress the grouping, and every quantity that does not depend on the draw
//     (lse_all, lse_ok, log_mass, status) comes from one shared routine.
//   * all floating point here is fp64.
//
// Parity pins for these functions live in tests/test_oracle_*.py.  The Philox
// uniform mapping and the counter layout are this build's own convention (the
// paper fixes no RNG): Philox itself is pinned by the published known-answer
// vectors, the layout only by the two independent implementations agreeing
// ("parity unpinned" for the layout).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

constexpr int ERR_ARG = -1, ERR_EMPTY = -2, ERR_TOKEN = -3, ERR_PREFIX = -4, ERR_UNSUPPORTED = -7;

// ---------------------------------------------------------------- edge table
// (parent node, token) -> child node.  Open addressing, linear probing.
struct EdgeTable {
    std::vector<uint64_t> key;
    std::vector<int32_t> val;
    uint64_t mask = 0;
    size_t count = 0;
    static constexpr uint64_t EMPTY = ~0ull;

    static uint64_t mix(uint64_t x) {
        x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ull;
        x ^= x >> 27; x *= 0x94d049bb133111ebull;
        x ^= x >> 31; return x;
    }
    void init(size_t cap_pow2) {
        key.assign(cap_pow2, EMPTY);
        val.assign(cap_pow2, -1);
        mask = cap_pow2 - 1;
        count = 0;
    }
    static uint64_t make_key(int32_t parent, int32_t token) {
        return (uint64_t(uint32_t(parent)) << 32) | uint32_t(token);
    }
    int32_t find(int32_t parent, int32_t token) const {
        uint64_t k = make_key(parent, token);
        for (uint64_t i = mix(k) & mask;; i = (i + 1) & mask) {
            if (key[i] == k) return val[i];
            if (key[i] == EMPTY) return -1;
        }
    }
    void grow() {
        std::vector<uint64_t> ok; ok.swap(key);
        std::vector<int32_t> ov; ov.swap(val);
        init(ok.size() * 2);
        for (size_t j = 0; j < ok.size(); ++j)
            if (ok[j] != EMPTY) put(ok[j], ov[j]);
    }
    void put(uint64_t k, int32_t v) {
        uint64_t i = mix(k) & mask;
        while (key[i] != EMPTY) i = (i + 1) & mask;
        key[i] = k; val[i] = v; ++count;
    }
    void insert(int32_t parent, int32_t token, int32_t child) {
        if ((count + 1) * 10 > key.size() * 6) grow();
        put(make_key(parent, token), child);
    }
};

// ---------------------------------------------------------------- prefix tree
struct Trie {
    int32_t V = 0;
    // node 0 is the root (the empty prefix).
    std::vector<int32_t> tok, first_child, next_sibling, lo, hi;
    std::vector<uint8_t> terminal;
    EdgeTable edges;
    // members in rank order
    std::vector<int32_t> sorted_tokens;
    std::vector<int64_t> sorted_off;
    int32_t l_max = 0;

    int32_t new_node(int32_t t) {
        tok.push_back(t); first_child.push_back(-1); next_sibling.push_back(-1);
        lo.push_back(-1); hi.push_back(-1); terminal.push_back(0);
        return int32_t(tok.size() - 1);
    }
    int32_t child(int32_t node, int32_t t) const { return edges.find(node, t); }

    int build(const int32_t* tokens, const int64_t* row_off, int64_t n_rows, int32_t vocab) {
        if (!tokens || !row_off || n_rows < 0 || vocab <= 0) return ERR_ARG;
        if (n_rows == 0) return ERR_EMPTY;
        V = vocab;
        edges.init(1 << 16);
        new_node(-1);
        for (int64_t r = 0; r < n_rows; ++r) {
            int64_t a = row_off[r], b = row_off[r + 1];
            if (b < a) return ERR_ARG;
            if (b == a) return ERR_EMPTY;
            int32_t node = 0;
            for (int64_t i = a; i < b; ++i) {
                int32_t t = tokens[i];
                if (t < 0 || t >= V) return ERR_TOKEN;
                int32_t c = child(node, t);
                if (c < 0) {
                    if (tok.size() >= size_t(std::numeric_limits<int32_t>::max())) return ERR_UNSUPPORTED;
                    c = new_node(t);
                    next_sibling[c] = first_child[node];
                    first_child[node] = c;
                    edges.insert(node, t, c);
                }
                node = c;
            }
            terminal[node] = 1;   // duplicates collapse here
        }
        // prefix-free: a member that has extensions is a proper prefix of another member
        for (size_t n = 0; n < tok.size(); ++n)
            if (terminal[n] && first_child[n] >= 0) return ERR_PREFIX;
        // put every child list in ascending token order
        std::vector<std::pair<int32_t, int32_t>> tmp;
        for (size_t n = 0; n < tok.size(); ++n) {
            if (first_child[n] < 0 || next_sibling[first_child[n]] < 0) continue;
            tmp.clear();
            for (int32_t c = first_child[n]; c >= 0; c = next_sibling[c]) tmp.push_back({tok[c], c});
            std::sort(tmp.begin(), tmp.end());
            first_child[n] = tmp[0].second;
            for (size_t i = 0; i < tmp.size(); ++i)
                next_sibling[tmp[i].second] = (i + 1 < tmp.size()) ? tmp[i + 1].second : -1;
        }
        // depth-first walk: rank the members, give every node its rank range
        struct Frame { int32_t node; int32_t next; };
        std::vector<Frame> stack;
        std::vector<int32_t> path;
        int32_t rank = 0;
        sorted_off.push_back(0);
        lo[0] = 0;
        stack.push_back({0, first_child[0]});
        while (!stack.empty()) {
            Frame& f = stack.back();
            if (f.next < 0) {
                hi[f.node] = rank;
                stack.pop_back();
                if (!path.empty()) path.pop_back();
                continue;
            }
            int32_t c = f.next;
            f.next = next_sibling[c];
            path.push_back(tok[c]);
            lo[c] = rank;
            if (terminal[c]) {
                sorted_tokens.insert(sorted_tokens.end(), path.begin(), path.end());
                sorted_off.push_back(int64_t(sorted_tokens.size()));
                l_max = std::max<int32_t>(l_max, int32_t(path.size()));
                ++rank;
            }
            stack.push_back({c, first_child[c]});
        }
        return 0;
    }

    // node reached by a prefix, or -1
    int32_t walk(const int32_t* prefix, int32_t len) const {
        int32_t node = 0;
        for (int32_t i = 0; i < len && node >= 0; ++i) {
            int32_t t = prefix[i];
            node = (t < 0 || t >= V) ? -1 : child(node, t);
        }
        return node;
    }
};

// ---------------------------------------------------------------- Philox4x32-10
// Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3" (2011).
void philox4x32_10(const uint32_t c_in[4], const uint32_t k_in[2], uint32_t out[4]) {
    uint32_t c[4] = {c_in[0], c_in[1], c_in[2], c_in[3]};
    uint32_t k[2] = {k_in[0], k_in[1]};
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }
        uint64_t p0 = uint64_t(0xD2511F53u) * c[0];
        uint64_t p1 = uint64_t(0xCD9E8D57u) * c[2];
        uint32_t n0 = uint32_t(p1 >> 32) ^ c[1] ^ k[0];
        uint32_t n1 = uint32_t(p1);
        uint32_t n2 = uint32_t(p0 >> 32) ^ c[3] ^ k[1];
        uint32_t n3 = uint32_t(p0);
        c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
    }
    out[0] = c[0]; out[1] = c[1]; out[2] = c[2]; out[3] = c[3];
}

// top 23 random bits k -> u = (2k+1) / 2^24: strictly inside (0,1), and both u and 1-u are
// exactly representable in fp32 (odd numerators below 2^24)
double uniform23(uint32_t r) { return (double(r >> 9) + 0.5) * (1.0 / 8388608.0); }

// Sampling works on groups of 8 consecutive token ids (group G = v >> 3); see step_row.
// domain 0: one uniform per (row, step, group).  Groups are spread over Philox counters so that the
// four words of one counter belong to groups 256 apart: counter word 0 = ((G>>10)<<8) | (G & 255),
// output word (G >> 8) & 3.  (Any bijection would do; this one is fixed by this build's convention.)
double group_uniform(uint64_t seed, uint32_t step, uint32_t row, uint32_t G) {
    uint32_t ctr[4] = {((G >> 10) << 8) | (G & 255u), step, row, 0u};
    uint32_t key[2] = {uint32_t(seed), uint32_t(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return uniform23(out[(G >> 8) & 3u]);
}
// domain 3: one uniform per (row, step, group) for the draw inside the winning group
double ingroup_uniform(uint64_t seed, uint32_t step, uint32_t row, uint32_t G) {
    uint32_t ctr[4] = {G, step, row, 3u};
    uint32_t key[2] = {uint32_t(seed), uint32_t(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return uniform23(out[0]);
}
// domain 1: one uniform per query for the K-way draw
double resample_uniform(uint64_t seed, uint32_t query) {
    uint32_t ctr[4] = {query, 0u, 0u, 1u};
    uint32_t key[2] = {uint32_t(seed), uint32_t(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return uniform23(out[0]);
}
// domain 2: one uniform per (query, candidate) for the accept test
double accept_uniform(uint64_t seed, uint32_t query, uint32_t k) {
    uint32_t ctr[4] = {query, k, 0u, 2u};
    uint32_t key[2] = {uint32_t(seed), uint32_t(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return uniform23(out[0]);
}

// domain 4: one uniform per (row, step) for the plain inverse-CDF sampler
double plain_uniform(uint64_t seed, uint32_t step, uint32_t row) {
    uint32_t ctr[4] = {0u, step, row, 4u};
    uint32_t key[2] = {uint32_t(seed), uint32_t(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return uniform23(out[0]);
}

double load_logit(const void* base, int dtype, int64_t idx) {
    if (dtype == 0) return double(static_cast<const float*>(base)[idx]);
    uint32_t bits = uint32_t(static_cast<const uint16_t*>(base)[idx]) << 16;   // bf16 -> f32
    float f;
    std::memcpy(&f, &bits, 4);
    return double(f);
}

constexpr double NEG_INF = -std::numeric_limits<double>::infinity();
constexpr double QNAN = std::numeric_limits<double>::quiet_NaN();

struct StepOut {
    int32_t token = -1, lo = -1, hi = -1;
    uint8_t done = 0, status = 0;
    double log_mass = QNAN, lse_all = QNAN, lse_ok = QNAN, logq = QNAN, logp = QNAN;
    double best = QNAN, second = QNAN, alt = QNAN;      // group scores: winner, runner-up, alt token's group
    double ingroup_gap = std::numeric_limits<double>::infinity();   // see step_row, stage (2)
    int32_t n_children = 0;
};

// log sum_v exp(z_v) with the maximum taken out first
struct Lse {
    double m = NEG_INF;
    std::vector<double> z;
    void add(double x) { z.push_back(x); if (x > m) m = x; }
    double value() const {
        if (z.empty()) return NEG_INF;
        bool any_nan = false;
        for (double x : z) any_nan |= std::isnan(x);
        if (any_nan) return QNAN;
        if (std::isinf(m)) return m;          // all -inf, or some +inf
        double s = 0.0;
        for (double x : z) s += std::exp(x - m);
        return m + std::log(s);
    }
};

// One decoding step of one row (Algorithm 1, lines 5-8) from the node its prefix reaches.
// plain = true draws the token with the plain inverse-CDF sampler instead of the two-stage one;
// nothing else differs.
// only: when given, the sorted token ids the mask is restricted to (the verified top-M candidates of
// Algorithm 2); a child whose token is not among them is treated as not allowed.  With no allowed
// token left the candidate has run into a dead end: status 1, no token, done.
StepOut step_row(const Trie& T, int32_t node, const void* logits, int dtype, int64_t base,
                 double inv_t, uint64_t seed, uint32_t step, uint32_t row, int32_t alt_token,
                 bool plain = false, const std::vector<int32_t>* only = nullptr) {
    StepOut o;
    if (node < 0) { o.status = 1; return o; }                 // prefix not in S
    if (T.first_child[node] < 0) { o.status = 8; o.done = 1; o.lo = T.lo[node]; o.hi = T.hi[node]; return o; }
    auto allowed = [&](int32_t c) { return !only || std::binary_search(only->begin(), only->end(), T.tok[c]); };

    Lse all;
    for (int32_t v = 0; v < T.V; ++v) all.add(load_logit(logits, dtype, base + v) * inv_t);
    o.lse_all = all.value();

    // Sampling from P.mask / |P.mask|_1 (Algorithm 1, line 7), exact, in two stages:
    //  (1) Gumbel-max over groups of 8 consecutive token ids (G = v >> 3): the score of a group is
    //      log(sum of e^{z_v} over its allowed tokens) - log(-log u_G); the largest score wins, the
    //      lowest group on an exact tie; NaN and -inf scores never win.  (The maximum of
    //      Gumbel-perturbed scores of a set of tokens is distributed as the perturbed log of their
    //      total mass, so the winning group is drawn with probability mass_G / total mass.)
    //  (2) inside the winning group, the smallest allowed token whose inclusive cumulative weight
    //      exceeds u' * mass_G (inverse CDF, tokens in ascending id).
    Lse ok;
    struct Member { int32_t child, tok; double z; };
    std::vector<Member> cur, win;
    int32_t cur_g = -1;
    double best = NEG_INF, second = NEG_INF;
    auto close_group = [&]() {
        if (cur.empty()) return;
        Lse mass;
        for (const Member& m : cur) mass.add(m.z);
        double u = group_uniform(seed, step, row, uint32_t(cur_g));
        double score = mass.value() + (-std::log(-std::log(u)));
        for (const Member& m : cur) if (m.tok == alt_token) o.alt = score;
        if (score > best) { second = best; best = score; win = cur; }
        else if (score > second) second = score;
        cur.clear();
    };
    int32_t first_allowed = -1;
    for (int32_t c = T.first_child[node]; c >= 0; c = T.next_sibling[c]) {
        if (!allowed(c)) continue;
        if (first_allowed < 0) first_allowed = c;
        ++o.n_children;
        int32_t v = T.tok[c];
        double z = load_logit(logits, dtype, base + v) * inv_t;
        ok.add(z);
        if ((v >> 3) != cur_g) { close_group(); cur_g = v >> 3; }
        cur.push_back({c, v, z});
    }
    close_group();
    if (first_allowed < 0) {                                   // top-M mode: none of the candidates is valid
        o.status = 1; o.done = 1; o.log_mass = NEG_INF; o.lse_ok = NEG_INF;
        return o;
    }
    int32_t best_child = first_allowed;                        // lowest id unless a group wins
    if (plain) {
        // Algorithm 1, line 7 as a textbook inverse CDF: weights e^{z_v - max} of the allowed
        // tokens in ascending id, the smallest token whose inclusive cumulative weight exceeds
        // u * total.  No groups, one uniform per (row, step).
        double zmax = NEG_INF, total = 0.0;
        for (int32_t c = T.first_child[node]; c >= 0; c = T.next_sibling[c])
            if (allowed(c)) zmax = std::max(zmax, load_logit(logits, dtype, base + T.tok[c]) * inv_t);
        if (std::isfinite(zmax)) {
            for (int32_t c = T.first_child[node]; c >= 0; c = T.next_sibling[c])
                if (allowed(c)) total += std::exp(load_logit(logits, dtype, base + T.tok[c]) * inv_t - zmax);
            if (std::isfinite(total) && total > 0.0) {
                const double target = plain_uniform(seed, step, row) * total;
                double cum = 0.0;
                for (int32_t c = T.first_child[node]; c >= 0; c = T.next_sibling[c]) {
                    if (!allowed(c)) continue;
                    cum += std::exp(load_logit(logits, dtype, base + T.tok[c]) * inv_t - zmax);
                    best_child = c;                            // the last allowed token if rounding leaves cum <= target
                    if (cum > target) break;
                }
            }
        }
    } else if (!win.empty()) {
        double zmax = NEG_INF, total = 0.0;
        for (const Member& m : win) if (m.z > zmax) zmax = m.z;
        std::vector<double> C(win.size());
        for (size_t i = 0; i < win.size(); ++i) { total += std::exp(win[i].z - zmax); C[i] = total; }
        size_t pick = 0;
        if (std::isfinite(total) && total > 0.0) {
            double target = ingroup_uniform(seed, step, row, uint32_t(win[0].tok >> 3)) * total;
            pick = win.size() - 1;
            for (size_t i = 0; i < win.size(); ++i) if (C[i] > target) { pick = i; break; }
            double below = pick > 0 ? C[pick - 1] : 0.0;
            o.ingroup_gap = std::min(std::fabs(target - below), std::fabs(C[pick] - target)) / total;
        }
        best_child = win[pick].child;
    }
    o.lse_ok = ok.value();
    o.log_mass = o.lse_ok - o.lse_all;
    if (!std::isfinite(o.lse_all)) o.status |= 4;
    if (!(o.lse_ok > NEG_INF) || !std::isfinite(o.lse_ok)) o.status |= 2;
    o.best = best; o.second = second;
    o.token = T.tok[best_child];
    double zt = load_logit(logits, dtype, base + o.token) * inv_t;
    o.logq = zt - o.lse_ok;
    o.logp = zt - o.lse_all;
    o.lo = T.lo[best_child];
    o.hi = T.hi[best_child];
    o.done = T.terminal[best_child];
    return o;
}

struct ResampleOut { int32_t idx; double logz; double u; double gap; uint8_t status; };

// Algorithm 1, line 22: index k with probability x_k / sum_j x_j, x = exp(logw).
ResampleOut resample_query(const double* logw, int32_t K, double u) {
    ResampleOut o{0, NEG_INF, u, std::numeric_limits<double>::infinity(), 0};
    double m = NEG_INF;
    for (int k = 0; k < K; ++k) {
        if (std::isnan(logw[k])) { o.status |= 4; continue; }
        if (logw[k] > m) m = logw[k];
    }
    if (!(m > NEG_INF) || std::isinf(m)) {       // no finite weight: uniform pick
        o.status |= 2;
        o.idx = std::min<int32_t>(K - 1, int32_t(std::floor(u * K)));
        o.logz = (m > 0) ? m : NEG_INF;
        return o;
    }
    std::vector<double> C(K);
    double acc = 0.0;
    for (int k = 0; k < K; ++k) {
        double w = std::isnan(logw[k]) ? 0.0 : std::exp(logw[k] - m);
        acc += w;
        C[k] = acc;
    }
    double target = u * C[K - 1];
    int32_t j = K - 1;
    for (int k = 0; k < K; ++k) if (C[k] > target) { j = k; break; }
    o.idx = j;
    o.logz = m + std::log(C[K - 1] / K);
    // distance from the threshold to the two boundaries of the chosen interval
    double below = (j > 0) ? C[j - 1] : 0.0;
    o.gap = std::min(std::fabs(target - below), std::fabs(C[j] - target)) / C[K - 1];
    return o;
}

template <class F>
void parallel_rows(int64_t n, int n_threads, F f) {
    if (n_threads <= 1 || n < 2) { for (int64_t i = 0; i < n; ++i) f(i); return; }
    std::vector<std::thread> pool;
    for (int t = 0; t < n_threads; ++t) {
        int64_t a = n * t / n_threads, b = n * (t + 1) / n_threads;
        pool.emplace_back([=] { for (int64_t i = a; i < b; ++i) f(i); });
    }
    for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

int oracle_build(const int32_t* tokens, const int64_t* row_off, int64_t n_rows, int32_t vocab,
                 void** out) {
    if (!out) return ERR_ARG;
    *out = nullptr;
    Trie* t = new Trie();
    int rc = t->build(tokens, row_off, n_rows, vocab);
    if (rc != 0) { delete t; return rc; }
    *out = t;
    return 0;
}

void oracle_free(void* h) { delete static_cast<Trie*>(h); }

// info[0]=N members, [1]=E table entries, [2]=l_max, [3]=tree nodes without the root
void oracle_info(const void* h, int64_t* info) {
    const Trie& T = *static_cast<const Trie*>(h);
    info[0] = int64_t(T.sorted_off.size()) - 1;
    info[1] = int64_t(T.sorted_tokens.size());
    info[2] = T.l_max;
    info[3] = int64_t(T.tok.size()) - 1;
}

void oracle_rows(const void* h, int32_t* tokens_out, int64_t* row_off_out) {
    const Trie& T = *static_cast<const Trie*>(h);
    std::memcpy(tokens_out, T.sorted_tokens.data(), T.sorted_tokens.size() * sizeof(int32_t));
    std::memcpy(row_off_out, T.sorted_off.data(), T.sorted_off.size() * sizeof(int64_t));
}

// Valid-set mask and member range of each prefix (Section 2.1).  mask is [n][W], W = ceil(V/32),
// token v <-> bit (v & 31) of word (v >> 5).  status 1 = prefix is not a prefix of any member.
void oracle_mask(const void* h, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                 int64_t n, uint32_t* mask, int32_t* lo, int32_t* hi, uint8_t* status) {
    const Trie& T = *static_cast<const Trie*>(h);
    int64_t W = (T.V + 31) / 32;
    for (int64_t i = 0; i < n; ++i) {
        uint32_t* m = mask + i * W;
        std::fill(m, m + W, 0u);
        int32_t node = T.walk(prefix + i * prefix_ld, prefix_len[i]);
        if (node < 0) { lo[i] = hi[i] = -1; status[i] = 1; continue; }
        lo[i] = T.lo[node]; hi[i] = T.hi[node]; status[i] = 0;
        for (int32_t c = T.first_child[node]; c >= 0; c = T.next_sibling[c])
            m[T.tok[c] >> 5] |= 1u << (T.tok[c] & 31);
    }
}

// Algorithm 2, lines 4-6, for n partial sequences with M candidate tokens each.  For candidate m of
// prefix i the row V_m = a + [t_m] is located in the sorted array X by a binary search for the
// smallest row that is not lexicographically smaller than V_m (index i_m, N when there is none;
// Section 3.2 "Parallel Verification"); t_m is valid iff V_m is a prefix of X_{i_m}.  valid is
// [n][M], row_index [n][M], mask [n][W] (line 6: bit t_m set iff valid; nullable).  A candidate
// outside [0, V) is invalid.
void oracle_verify(const void* h, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                   int64_t n, const int32_t* cand, int32_t M, uint8_t* valid, int32_t* row_index,
                   uint32_t* mask) {
    const Trie& T = *static_cast<const Trie*>(h);
    const int64_t N = int64_t(T.sorted_off.size()) - 1;
    const int64_t W = (T.V + 31) / 32;
    std::vector<int64_t> rows(N);
    for (int64_t j = 0; j < N; ++j) rows[j] = j;
    std::vector<int32_t> Vm;
    for (int64_t i = 0; i < n; ++i) {
        if (mask) std::fill(mask + i * W, mask + (i + 1) * W, 0u);
        for (int32_t m = 0; m < M; ++m) {
            const int32_t t = cand[i * M + m];
            Vm.assign(prefix + i * prefix_ld, prefix + i * prefix_ld + prefix_len[i]);
            Vm.push_back(t);
            auto it = std::lower_bound(rows.begin(), rows.end(), Vm, [&](int64_t j, const std::vector<int32_t>& v) {
                return std::lexicographical_compare(T.sorted_tokens.begin() + T.sorted_off[j],
                                                    T.sorted_tokens.begin() + T.sorted_off[j + 1], v.begin(), v.end());
            });
            const int64_t im = it - rows.begin();
            bool ok = false;
            if (im < N && t >= 0 && t < T.V) {
                const int64_t a = T.sorted_off[im], b = T.sorted_off[im + 1];
                ok = (b - a) >= int64_t(Vm.size()) && std::equal(Vm.begin(), Vm.end(), T.sorted_tokens.begin() + a);
            }
            valid[i * M + m] = ok ? 1 : 0;
            row_index[i * M + m] = int32_t(im);
            if (ok && mask) mask[i * W + (t >> 5)] |= 1u << (t & 31);
        }
    }
}

// Algorithm 2, line 3: the M tokens of highest probability of one row, i.e. of largest logit.
// Equal logits are common (bf16 has few distinct values): the lower token id comes first; NaN
// logits come last.  Returned in ascending token id.
std::vector<int32_t> top_m_row(const void* logits, int dtype, int64_t base, int32_t V, int32_t M) {
    std::vector<int32_t> idx(V);
    for (int32_t v = 0; v < V; ++v) idx[v] = v;
    auto key = [&](int32_t v) { double z = load_logit(logits, dtype, base + v); return std::isnan(z) ? NEG_INF : z; };
    auto nan_last = [&](int32_t v) { return std::isnan(load_logit(logits, dtype, base + v)) ? 1 : 0; };
    std::stable_sort(idx.begin(), idx.end(), [&](int32_t a, int32_t b) {
        if (nan_last(a) != nan_last(b)) return nan_last(a) < nan_last(b);
        return key(a) > key(b);
    });
    idx.resize(std::min(M, V));
    std::sort(idx.begin(), idx.end());
    return idx;
}

// Algorithm 2, lines 4-5 for one candidate: V_m = a + [t] is located in the sorted array by binary
// search (the smallest row not smaller than V_m); t is valid iff V_m is a prefix of that row.
bool verify_candidate(const Trie& T, const int32_t* prefix, int32_t len, int32_t t) {
    const int64_t N = int64_t(T.sorted_off.size()) - 1;
    if (t < 0 || t >= T.V) return false;
    std::vector<int32_t> Vm(prefix, prefix + len);
    Vm.push_back(t);
    int64_t a = 0, b = N;
    while (a < b) {
        const int64_t mid = (a + b) / 2;
        const bool smaller = std::lexicographical_compare(T.sorted_tokens.begin() + T.sorted_off[mid],
                                                          T.sorted_tokens.begin() + T.sorted_off[mid + 1],
                                                          Vm.begin(), Vm.end());
        if (smaller) a = mid + 1; else b = mid;
    }
    if (a >= N) return false;
    const int64_t r0 = T.sorted_off[a], r1 = T.sorted_off[a + 1];
    return (r1 - r0) >= int64_t(Vm.size()) && std::equal(Vm.begin(), Vm.end(), T.sorted_tokens.begin() + r0);
}

// Top-M candidates of n rows (Algorithm 2, line 3), ascending token id per row; cand is [n][M].
void oracle_topm(const void* logits, int dtype, int64_t ld, int64_t n, int32_t V, int32_t M, int32_t* cand) {
    for (int64_t i = 0; i < n; ++i) {
        std::vector<int32_t> c = top_m_row(logits, dtype, i * ld, V, M);
        for (int32_t m = 0; m < M; ++m) cand[i * M + m] = m < int32_t(c.size()) ? c[m] : -1;
    }
}

// One decoding step in the paper's top-M mode (Algorithm 1, lines 5-8 with the mask of Algorithm 2,
// lines 3-6): the M most probable tokens are the candidates, each is verified against the sorted
// array, the token is drawn among the verified ones and the importance score is multiplied by their
// probability mass.  A row none of whose candidates is valid has reached a dead end (it will fail
// Algorithm 1's test "a in S"): status 1, token -1, done, log_mass = -inf.  Outputs as for
// oracle_step; n_valid[i] is the number of verified candidates.
void oracle_step_topm(const void* h, const void* logits, int dtype, int64_t ld, int64_t n, int32_t M,
                      float inv_temperature, uint64_t seed, uint32_t step, const int64_t* row_ids,
                      const int32_t* prefix, int32_t prefix_ld, const int32_t* depth, const uint8_t* done,
                      const int32_t* alt_token,
                      int32_t* token, int32_t* lo, int32_t* hi, uint8_t* done_out,
                      double* log_mass, double* lse_all, double* lse_ok, double* logq, double* logp,
                      double* best_score, double* second_score, double* alt_score, double* ingroup_gap,
                      int32_t* n_valid, uint8_t* status, int n_threads) {
    const Trie& T = *static_cast<const Trie*>(h);
    parallel_rows(n, n_threads, [&](int64_t i) {
        StepOut o;
        if (done && done[i]) {
            o.status = 8; o.done = 1;
        } else {
            const int32_t* pre = prefix + i * prefix_ld;
            int32_t node = T.walk(pre, depth[i]);
            uint32_t row = uint32_t(row_ids ? row_ids[i] : i);
            std::vector<int32_t> cand = top_m_row(logits, dtype, i * ld, T.V, M), ok;
            for (int32_t t : cand) if (verify_candidate(T, pre, depth[i], t)) ok.push_back(t);
            o = step_row(T, node, logits, dtype, i * ld, double(inv_temperature), seed, step, row,
                         alt_token ? alt_token[i] : -1, false, &ok);
        }
        token[i] = o.token; lo[i] = o.lo; hi[i] = o.hi; done_out[i] = o.done;
        log_mass[i] = o.log_mass; lse_all[i] = o.lse_all; lse_ok[i] = o.lse_ok;
        logq[i] = o.logq; logp[i] = o.logp;
        best_score[i] = o.best; second_score[i] = o.second;
        if (alt_score) alt_score[i] = o.alt;
        if (ingroup_gap) ingroup_gap[i] = o.ingroup_gap;
        if (n_valid) n_valid[i] = o.n_children;
        status[i] = o.status;
    });
}

// One decoding step for n rows.  Row i's prefix is prefix[i*prefix_ld .. +depth[i]); its logits are
// logits[i*ld .. +V); its RNG row index is row_ids[i] (i when row_ids is null).  Rows with done[i]
// != 0 are skipped (token -1, status 8).  Every output array has n entries; alt_token is optional:
// alt_score[i] is this oracle's perturbed score of the group of alt_token[i] (NaN if that token is
// not allowed); best/second are the winning and runner-up group scores; ingroup_gap[i] is the
// distance of the in-group threshold to the nearest boundary of the chosen token's interval, as a
// fraction of the group's mass (for near-tie accounting).
void oracle_step(const void* h, const void* logits, int dtype, int64_t ld, int64_t n,
                 float inv_temperature, uint64_t seed, uint32_t step, const int64_t* row_ids,
                 const int32_t* prefix, int32_t prefix_ld, const int32_t* depth, const uint8_t* done,
                 const int32_t* alt_token,
                 int32_t* token, int32_t* lo, int32_t* hi, uint8_t* done_out,
                 double* log_mass, double* lse_all, double* lse_ok, double* logq, double* logp,
                 double* best_score, double* second_score, double* alt_score, double* ingroup_gap,
                 int32_t* n_children, uint8_t* status, int n_threads) {
    const Trie& T = *static_cast<const Trie*>(h);
    parallel_rows(n, n_threads, [&](int64_t i) {
        StepOut o;
        if (done && done[i]) {
            o.status = 8; o.done = 1;
        } else {
            int32_t node = T.walk(prefix + i * prefix_ld, depth[i]);
            uint32_t row = uint32_t(row_ids ? row_ids[i] : i);
            o = step_row(T, node, logits, dtype, i * ld, double(inv_temperature), seed, step, row,
                         alt_token ? alt_token[i] : -1);
        }
        token[i] = o.token; lo[i] = o.lo; hi[i] = o.hi; done_out[i] = o.done;
        log_mass[i] = o.log_mass; lse_all[i] = o.lse_all; lse_ok[i] = o.lse_ok;
        logq[i] = o.logq; logp[i] = o.logp;
        best_score[i] = o.best; second_score[i] = o.second;
        if (alt_score) alt_score[i] = o.alt;
        if (ingroup_gap) ingroup_gap[i] = o.ingroup_gap;
        if (n_children) n_children[i] = o.n_children;
        status[i] = o.status;
    });
}

// The same step with the plain sampler (inverse CDF over the allowed tokens, one uniform per row
// and step; see the top of this file).  Arguments as for oracle_step; the outputs that describe the
// two-stage draw are absent.
void oracle_step_plain(const void* h, const void* logits, int dtype, int64_t ld, int64_t n,
                       float inv_temperature, uint64_t seed, uint32_t step, const int64_t* row_ids,
                       const int32_t* prefix, int32_t prefix_ld, const int32_t* depth, const uint8_t* done,
                       int32_t* token, int32_t* lo, int32_t* hi, uint8_t* done_out,
                       double* log_mass, double* lse_all, double* lse_ok, double* logq, double* logp,
                       uint8_t* status, int n_threads) {
    const Trie& T = *static_cast<const Trie*>(h);
    parallel_rows(n, n_threads, [&](int64_t i) {
        StepOut o;
        if (done && done[i]) {
            o.status = 8; o.done = 1;
        } else {
            int32_t node = T.walk(prefix + i * prefix_ld, depth[i]);
            uint32_t row = uint32_t(row_ids ? row_ids[i] : i);
            o = step_row(T, node, logits, dtype, i * ld, double(inv_temperature), seed, step, row, -1, true);
        }
        token[i] = o.token; lo[i] = o.lo; hi[i] = o.hi; done_out[i] = o.done;
        log_mass[i] = o.log_mass; lse_all[i] = o.lse_all; lse_ok[i] = o.lse_ok;
        logq[i] = o.logq; logp[i] = o.logp; status[i] = o.status;
    });
}

// K-way importance draw for B queries (Algorithm 1, line 22).  logw is [B][K] fp32 (the bytes the
// CUDA path holds), widened to fp64 here.  query_ids (nullable) are the RNG query indices.
// gap[b] = distance of the threshold to the nearest boundary of the chosen interval, as a fraction
// of the total weight (for near-tie accounting).
void oracle_resample(const float* logw, int32_t B, int32_t K, uint64_t seed, const int64_t* query_ids,
                     int32_t* idx, double* logz, double* u_out, double* gap, uint8_t* status) {
    std::vector<double> lw(K);
    for (int32_t b = 0; b < B; ++b) {
        for (int k = 0; k < K; ++k) lw[k] = double(logw[int64_t(b) * K + k]);
        double u = resample_uniform(seed, uint32_t(query_ids ? query_ids[b] : b));
        ResampleOut o = resample_query(lw.data(), K, u);
        idx[b] = o.idx; logz[b] = o.logz; status[b] = o.status;
        if (u_out) u_out[b] = o.u;
        if (gap) gap[b] = o.gap;
    }
}

// Accept test of Algorithm 1, line 16, applied to K finished candidates per query in order:
// first k with x_k > eps_k, i.e. logw_k > log(eps_k); -1 when all K are rejected.
void oracle_accept(const float* logw, int32_t B, int32_t K, uint64_t seed, const int64_t* query_ids,
                   int32_t* first_accepted) {
    for (int32_t b = 0; b < B; ++b) {
        first_accepted[b] = -1;
        uint32_t q = uint32_t(query_ids ? query_ids[b] : b);
        for (int32_t k = 0; k < K; ++k) {
            double eps = accept_uniform(seed, q, uint32_t(k));
            if (double(logw[int64_t(b) * K + k]) > std::log(eps)) { first_accepted[b] = k; break; }
        }
    }
}

// Algorithm 1, lines 11-22, on 2K finished candidates per query (logw is [B][2K]): candidates
// 0..K-1 go through the accept test in order (lines 12-20: return the first with x > eps); when
// all K are rejected, one of the K fresh candidates K..2K-1 is drawn with probability
// x_k / sum_j x_j (line 22).  choice[b] is the column returned, first_accepted[b] the accepted
// candidate or -1, logz/gap/status describe the K-way draw over the fresh candidates (computed for
// every query, used only after K rejections).
void oracle_accept_resample(const float* logw, int32_t B, int32_t K, uint64_t seed, const int64_t* query_ids,
                            int32_t* choice, int32_t* first_accepted, double* logz, double* gap, uint8_t* status) {
    std::vector<double> lw(K);
    for (int32_t b = 0; b < B; ++b) {
        const float* w = logw + int64_t(b) * 2 * K;
        uint32_t q = uint32_t(query_ids ? query_ids[b] : b);
        int32_t first = -1;
        for (int32_t k = 0; k < K && first < 0; ++k)
            if (double(w[k]) > std::log(accept_uniform(seed, q, uint32_t(k)))) first = k;
        for (int k = 0; k < K; ++k) lw[k] = double(w[K + k]);
        ResampleOut o = resample_query(lw.data(), K, resample_uniform(seed, q));
        first_accepted[b] = first;
        choice[b] = first >= 0 ? first : K + o.idx;
        logz[b] = o.logz; status[b] = o.status;
        if (gap) gap[b] = o.gap;
    }
}

// Free-running decode of B queries x K candidates under a first-order Markov language model given
// as a table: logits of the next token after token p are Z[p*V .. +V) (fp32); the first step uses
// the query's context token.  Runs Algorithm 1's SampleCandidate for every (query, candidate) and
// then the K-way draw.  seq is [B][K][l_max] (-1 padded), logw_out [B][K] fp64, logw32 [B][K] the
// same rounded step by step to fp32 (what a caller holding fp32 state would have).
int oracle_decode_markov(const void* h, const float* Z, const int32_t* ctx, int32_t B, int32_t K,
                         float inv_temperature, uint64_t seed, int64_t query_base,
                         int32_t* seq, int32_t* seq_len, double* logw_out, float* logw32,
                         int32_t* idx, double* logz, int n_threads) {
    const Trie& T = *static_cast<const Trie*>(h);
    int32_t L = T.l_max;
    int64_t R = int64_t(B) * K;
    parallel_rows(R, n_threads, [&](int64_t r) {
        int32_t b = int32_t(r / K);
        int32_t* s = seq + r * L;
        std::fill(s, s + L, -1);
        int32_t node = 0, prev = ctx[b], len = 0;
        double lw = 0.0;
        float lw32 = 0.0f;
        uint32_t row = uint32_t(query_base * K + r);
        while (T.first_child[node] >= 0) {
            StepOut o = step_row(T, node, Z, 0, int64_t(prev) * T.V, double(inv_temperature), seed,
                                 uint32_t(len), row, -1);
            lw += o.log_mass;
            lw32 = float(double(lw32) + o.log_mass);
            s[len++] = o.token;
            node = T.child(node, o.token);
            prev = o.token;
        }
        seq_len[r] = len; logw_out[r] = lw; logw32[r] = lw32;
    });
    std::vector<double> lw(K);
    for (int32_t b = 0; b < B; ++b) {
        for (int k = 0; k < K; ++k) lw[k] = double(logw32[int64_t(b) * K + k]);
        ResampleOut o = resample_query(lw.data(), K, resample_uniform(seed, uint32_t(query_base + b)));
        idx[b] = o.idx; logz[b] = o.logz;
    }
    return 0;
}

void oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}

double oracle_group_uniform(uint64_t seed, uint32_t step, uint32_t row, uint32_t G) {
    return group_uniform(seed, step, row, G);
}
double oracle_ingroup_uniform(uint64_t seed, uint32_t step, uint32_t row, uint32_t G) {
    return ingroup_uniform(seed, step, row, G);
}
double oracle_plain_uniform(uint64_t seed, uint32_t step, uint32_t row) { return plain_uniform(seed, step, row); }
double oracle_resample_uniform(uint64_t seed, uint32_t query) { return resample_uniform(seed, query); }
double oracle_accept_uniform(uint64_t seed, uint32_t query, uint32_t k) { return accept_uniform(seed, query, k); }

}  // extern "C"
