// Host-side setup: online suffix-automaton construction (Section 5.4.3: built incrementally,
// token by token, linear in the context length) and flattening to CSR + the packed device image.
// The builder itself lives in sam_builder.h.
#include <algorithm>
#include <cstring>
#include <new>
#include <utility>

#include "sam_builder.h"
#include "sam_index.h"

namespace samb200 {

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
            if (d >= 3) wide += (d <= kSortedRowMax) ? d : (int64_t(1) << hash_log2cap(static_cast<int32_t>(d), 2));
        }
        if (wide >= (int64_t(1) << 31) - 64) return SAM_ERR_TOO_LARGE;   // row offsets are 32-bit
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
        } else if (d >= 3 && d <= kSortedRowMax) {
            r.e[0] = static_cast<int32_t>(w);
            for (int64_t k = lo; k < hi; ++k, ++w) { wide[w].tok = idx.edge_tok[k]; wide[w].dst = idx.edge_dst[k]; }
        } else if (d > kSortedRowMax) {
            const int32_t lc = hash_log2cap(static_cast<int32_t>(d), 2);
            const int64_t cap = int64_t(1) << lc;
            Edge* row = wide + w;
            for (int64_t k = 0; k < cap; ++k) row[k] = Edge{-1, -1};
            for (int64_t k = lo; k < hi; ++k) {
                uint32_t at = hash_slot(idx.edge_tok[k], lc);
                while (row[at].tok >= 0) at = (at + 1) & static_cast<uint32_t>(cap - 1);
                row[at] = Edge{idx.edge_tok[k], idx.edge_dst[k]};
            }
            r.e[0] = static_cast<int32_t>(w);
            r.e[1] = lc;
            w += cap;
        }
        rec[s] = r;
    }
    for (int64_t t = 0; t < idx.layout.root_span; ++t) root_dst[t] = -1;
    for (int64_t k = idx.row_ptr[0]; k < idx.row_ptr[1]; ++k)
        if (idx.edge_tok[k] >= 0) root_dst[idx.edge_tok[k]] = idx.edge_dst[k];
}

}  // namespace samb200
