// Host-side setup: online suffix-automaton construction (Section 5.4.3: built incrementally,
// token by token, linear in the context length) and flattening to CSR + the packed device image.
//
// Container strategy: every transition is a node of one global pool, chained per source
// state (newest first).  States with few transitions are searched by walking their chain;
// once a state has more than kHeavy transitions all of them are also indexed in one
// open-addressing hash table keyed by (state, token).  Rows are sorted by token id only
// when the automaton is flattened.
#include <algorithm>
#include <cstring>
#include <new>
#include <utility>

#include "sam_index.h"

namespace samb200 {
namespace {

constexpr int32_t kHeavy = 6;
constexpr uint64_t kEmpty = ~0ull;

struct Builder {
    std::vector<int32_t> len, link, fpos, head, deg;
    std::vector<int32_t> e_tok, e_dst, e_next;
    std::vector<uint64_t> hkey;
    std::vector<int32_t> hval;
    uint64_t hmask = 0;
    int64_t hcount = 0;

    static uint64_t key_of(int32_t s, int32_t c) {
        return (static_cast<uint64_t>(static_cast<uint32_t>(s)) << 32) | static_cast<uint32_t>(c);
    }
    static uint64_t mix(uint64_t k) {
        k ^= k >> 31;
        k *= 0x9E3779B97F4A7C15ull;
        k ^= k >> 29;
        k *= 0xBF58476D1CE4E5B9ull;
        k ^= k >> 32;
        return k;
    }
    void hash_alloc(uint64_t size) {
        hkey.assign(size, kEmpty);
        hval.assign(size, -1);
        hmask = size - 1;
    }
    void hash_put_raw(uint64_t k, int32_t e) {
        uint64_t i = mix(k) & hmask;
        while (hkey[i] != kEmpty) i = (i + 1) & hmask;
        hkey[i] = k;
        hval[i] = e;
    }
    void hash_put(int32_t s, int32_t c, int32_t e) {
        if (static_cast<uint64_t>(hcount + 1) * 2 > hmask + 1) {
            std::vector<uint64_t> ok;
            std::vector<int32_t> ov;
            ok.swap(hkey);
            ov.swap(hval);
            hash_alloc((hmask + 1) * 2);
            for (size_t i = 0; i < ok.size(); ++i)
                if (ok[i] != kEmpty) hash_put_raw(ok[i], ov[i]);
        }
        hash_put_raw(key_of(s, c), e);
        ++hcount;
    }
    int32_t hash_get(int32_t s, int32_t c) const {
        const uint64_t k = key_of(s, c);
        uint64_t i = mix(k) & hmask;
        while (hkey[i] != kEmpty) {
            if (hkey[i] == k) return hval[i];
            i = (i + 1) & hmask;
        }
        return -1;
    }

    int32_t new_state(int32_t l, int32_t lk, int32_t fp) {
        len.push_back(l);
        link.push_back(lk);
        fpos.push_back(fp);
        head.push_back(-1);
        deg.push_back(0);
        return static_cast<int32_t>(len.size() - 1);
    }
    // pool index of the transition (s, c), or -1
    int32_t find(int32_t s, int32_t c) const {
        if (deg[s] > kHeavy) return hash_get(s, c);
        for (int32_t e = head[s]; e >= 0; e = e_next[e])
            if (e_tok[e] == c) return e;
        return -1;
    }
    void add(int32_t s, int32_t c, int32_t d) {
        const int32_t e = static_cast<int32_t>(e_tok.size());
        e_tok.push_back(c);
        e_dst.push_back(d);
        e_next.push_back(head[s]);
        head[s] = e;
        const int32_t n = ++deg[s];
        if (n == kHeavy + 1) {
            for (int32_t x = head[s]; x >= 0; x = e_next[x]) hash_put(s, e_tok[x], x);
        } else if (n > kHeavy + 1) {
            hash_put(s, c, e);
        }
    }

    void extend(int32_t c, int32_t pos, int32_t& last) {
        const int32_t cur = new_state(len[last] + 1, -1, pos);
        int32_t p = last;
        int32_t e = -1;
        while (p != -1 && (e = find(p, c)) < 0) {
            add(p, c, cur);
            p = link[p];
        }
        if (p == -1) {
            link[cur] = 0;
        } else {
            const int32_t q = e_dst[e];
            if (len[p] + 1 == len[q]) {
                link[cur] = q;
            } else {
                const int32_t clone = new_state(len[p] + 1, link[q], fpos[q]);
                for (int32_t x = head[q]; x >= 0; x = e_next[x]) add(clone, e_tok[x], e_dst[x]);
                while (p != -1) {
                    const int32_t ex = find(p, c);
                    if (ex < 0 || e_dst[ex] != q) break;
                    e_dst[ex] = clone;
                    p = link[p];
                }
                link[q] = clone;
                link[cur] = clone;
            }
        }
        last = cur;
    }
};

}  // namespace

int build_index(const int32_t* corpus, int64_t n, const int32_t* seps, int32_t n_sep, sam_index* out) {
    try {
        Builder b;
        const size_t rs = static_cast<size_t>(n) + static_cast<size_t>(n) / 2 + 16;
        b.len.reserve(rs); b.link.reserve(rs); b.fpos.reserve(rs); b.head.reserve(rs); b.deg.reserve(rs);
        const size_t re = static_cast<size_t>(n) * 2 + static_cast<size_t>(n) / 4 + 16;
        b.e_tok.reserve(re); b.e_dst.reserve(re); b.e_next.reserve(re);
        b.hash_alloc(1u << 16);
        b.new_state(0, -1, -1);
        int32_t last = 0;
        for (int64_t i = 0; i < n; ++i) b.extend(corpus[i], static_cast<int32_t>(i), last);

        const int64_t S = static_cast<int64_t>(b.len.size());
        const int64_t E = static_cast<int64_t>(b.e_tok.size());
        out->len.swap(b.len);
        out->link.swap(b.link);
        out->firstpos.swap(b.fpos);
        { std::vector<uint64_t>().swap(b.hkey); std::vector<int32_t>().swap(b.hval); }
        out->row_ptr.resize(static_cast<size_t>(S) + 1);
        out->edge_tok.resize(static_cast<size_t>(E));
        out->edge_dst.resize(static_cast<size_t>(E));
        int64_t off = 0;
        std::vector<std::pair<int32_t, int32_t>> tmp;
        for (int64_t s = 0; s < S; ++s) {
            out->row_ptr[s] = off;
            const int32_t d = b.deg[s];
            if (d == 1) {
                out->edge_tok[off] = b.e_tok[b.head[s]];
                out->edge_dst[off] = b.e_dst[b.head[s]];
            } else if (d > 1) {
                tmp.clear();
                for (int32_t x = b.head[s]; x >= 0; x = b.e_next[x]) tmp.emplace_back(b.e_tok[x], b.e_dst[x]);
                std::sort(tmp.begin(), tmp.end());
                for (int32_t k = 0; k < d; ++k) {
                    out->edge_tok[off + k] = tmp[k].first;
                    out->edge_dst[off + k] = tmp[k].second;
                }
            }
            off += d;
        }
        out->row_ptr[S] = off;
        out->corpus.assign(corpus, corpus + n);
        out->seps.assign(seps, seps + n_sep);

        // device layout
        DeviceLayout& L = out->layout;
        L.n_states = S;
        L.n_corpus = n;
        int64_t wide = 0;
        for (int64_t s = 1; s < S; ++s) {
            const int64_t d = out->row_ptr[s + 1] - out->row_ptr[s];
            if (d >= 3) wide += d;
        }
        L.n_wide_edges = wide;
        int64_t span = 0;  // dense root table covers token ids [0, span)
        for (int64_t k = out->row_ptr[0]; k < out->row_ptr[1]; ++k)
            if (out->edge_tok[k] >= 0) span = std::max<int64_t>(span, static_cast<int64_t>(out->edge_tok[k]) + 1);
        L.root_span = span;
        auto up = [](int64_t x) { return (x + 255) & ~int64_t(255); };
        L.rec_off = 0;
        L.edge_off = up(L.rec_off + S * static_cast<int64_t>(sizeof(StateRec)));
        L.root_off = up(L.edge_off + wide * static_cast<int64_t>(sizeof(Edge)));
        L.corpus_off = up(L.root_off + span * 4);
        L.total = up(L.corpus_off + n * 4);
        return SAM_OK;
    } catch (const std::bad_alloc&) {
        return SAM_ERR_NOMEM;
    }
}

void pack_records(const sam_index& idx, StateRec* rec, Edge* wide, int32_t* root_dst) {
    const int64_t S = idx.layout.n_states;
    int64_t w = 0;
    for (int64_t s = 0; s < S; ++s) {
        const int64_t lo = idx.row_ptr[s], hi = idx.row_ptr[s + 1];
        const int64_t d = hi - lo;
        StateRec r;
        r.len = idx.len[s];
        r.link = idx.link[s];
        r.firstpos = idx.firstpos[s];
        r.deg = static_cast<int32_t>(d);
        r.e[0] = r.e[1] = r.e[2] = r.e[3] = -1;
        if (s == 0) {
            // dense table filled below
        } else if (d == 1 || d == 2) {
            r.e[0] = idx.edge_tok[lo];
            r.e[1] = idx.edge_dst[lo];
            if (d == 2) { r.e[2] = idx.edge_tok[lo + 1]; r.e[3] = idx.edge_dst[lo + 1]; }
        } else if (d >= 3) {
            r.e[0] = static_cast<int32_t>(w);
            for (int64_t k = lo; k < hi; ++k, ++w) { wide[w].tok = idx.edge_tok[k]; wide[w].dst = idx.edge_dst[k]; }
        }
        rec[s] = r;
    }
    for (int64_t t = 0; t < idx.layout.root_span; ++t) root_dst[t] = -1;
    for (int64_t k = idx.row_ptr[0]; k < idx.row_ptr[1]; ++k)
        if (idx.edge_tok[k] >= 0) root_dst[idx.edge_tok[k]] = idx.edge_dst[k];
}

}  // namespace samb200
