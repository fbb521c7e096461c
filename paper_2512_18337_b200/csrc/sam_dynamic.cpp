// Growing index: the automaton keeps absorbing tokens after it was built (Section 5.4.2: verified
// tokens are inserted so that the index follows the growing context) and a builder thread does the
// construction off the decoding path (Section 5.4.3: construction is offloaded to a child thread
// that serves a waiting queue; until an update is ready, drafting goes on with what is there).
//
// The builder thread owns the automaton.  For every chunk of tokens it takes from the queue it runs
// the online construction, then packs what changed - records of touched states, rewritten wide
// rows, changed root entries, the appended text - into a Delta that the caller's thread later
// copies to the device (sam_sync).  Wide rows get power-of-two capacity so that most rewrites happen
// in place; when the wide area is exhausted all rows are laid out afresh and the next update is a
// full image.
#include <algorithm>
#include <condition_variable>
#include <climits>
#include <cstdlib>
#include <cstring>
#include <deque>
#include <mutex>
#include <new>
#include <atomic>
#include <thread>
#include <unordered_map>

#include "sam_builder.h"
#include "sam_index.h"

namespace samb200 {

struct DynIndex {
    sam_index* owner = nullptr;
    Builder b;
    int32_t last = 0;
    std::vector<int32_t> corpus;
    int64_t max_tokens = 0, s_cap = 0, w_cap = 0, span_cap = 0;
    std::vector<int32_t> wide_off, wide_cap;   // per state: row offset / capacity in the device's wide array (-1 / 0: none)
    std::vector<int32_t> packed_deg;           // per state: transitions its wide row held when it was last packed
    std::vector<Edge> mirror;                  // host copy of the device's wide array (rows sorted by token)
    int64_t w_used = 0;
    std::atomic<int64_t> relayout_every{0};    // > 0: lay the wide rows out afresh at every k-th update (sam_growing_set_relayout_every)
    int64_t updates_packed = 0;

    std::thread worker;
    std::mutex mu;
    std::condition_variable cv_work, cv_idle;
    std::deque<std::vector<int32_t>> inbox;
    std::deque<Delta> ready;
    bool stop = false, busy = false;
    int64_t queued = 0, built = 0;
    int error = SAM_OK;
};

namespace {

int32_t pow2_at_least(int32_t d) {
    int32_t c = 4;
    while (c < d) c <<= 1;
    return c;
}

// Appends "edges [first, first + count) of the row at `off` changed" to the delta (nothing when segs is null).
void note_segment(DynIndex& D, Delta* out, int64_t off, int64_t first, int64_t count) {
    if (!out || count <= 0) return;
    WideSeg g;
    g.dst_off = off + first;
    g.src_off = static_cast<int64_t>(out->seg_edges.size());
    g.len = static_cast<int32_t>(count);
    out->segs.push_back(g);
    const Edge* row = D.mirror.data() + off + first;
    out->seg_edges.insert(out->seg_edges.end(), row, row + count);
}

bool place_row(DynIndex& D, int32_t s, int32_t cap) {
    if (D.w_used + cap > D.w_cap) return false;
    D.wide_off[s] = static_cast<int32_t>(D.w_used);
    D.wide_cap[s] = cap;
    D.w_used += cap;
    if (D.mirror.size() < static_cast<size_t>(D.w_used)) D.mirror.resize(static_cast<size_t>(D.w_used), Edge{-1, -1});
    return true;
}

// Slot of token tok in the hash row (its own slot, or the empty one where it would go).
uint32_t hash_find(const Edge* row, int32_t lc, int32_t tok) {
    const uint32_t mask = (1u << lc) - 1u;
    uint32_t at = hash_slot(tok, lc);
    while (row[at].tok >= 0 && row[at].tok != tok) at = (at + 1) & mask;
    return at;
}

// Record of state s (not the root).  Wide rows live in the host mirror of the device's wide array.
// Up to kSortedRowMax transitions a row is a sorted array in a power-of-two slot: the transitions added
// since the last packing (the newest nodes of the state's chain) are merged in, redirected ones patched.
// Beyond that it is a hash table: a new transition is one slot written, a redirected one one slot
// patched; the table moves (and is sent whole) only when it is half full.  What differs from the device's
// copy is appended to `out` (null: nothing is recorded, the caller sends everything).
// Returns false when the wide area is exhausted.
bool pack_state(DynIndex& D, int32_t s, StateRec* r, const std::pair<int32_t, int32_t>* redir, size_t n_redir,
                std::vector<std::pair<int32_t, int32_t>>& tmp, Delta* out) {
    const Builder& b = D.b;
    r->len = b.len[s];
    r->link = b.link[s];
    r->firstpos = b.fpos[s];
    r->deg = b.deg[s];
    r->e[0] = r->e[1] = r->e[2] = r->e[3] = -1;
    const int32_t d = b.deg[s];
    if (d <= 2) {
        // the common case by far: read the one or two chain nodes directly
        if (d >= 1) {
            const int32_t x0 = b.head[s];
            if (d == 1) {
                r->e[0] = b.e_tok[x0];
                r->e[1] = b.e_dst[x0];
            } else {
                const int32_t x1 = b.e_next[x0];
                const bool swap = b.e_tok[x1] < b.e_tok[x0];
                const int32_t lo = swap ? x1 : x0, hi = swap ? x0 : x1;
                r->e[0] = b.e_tok[lo]; r->e[1] = b.e_dst[lo];
                r->e[2] = b.e_tok[hi]; r->e[3] = b.e_dst[hi];
            }
        }
        return true;
    }
    if (static_cast<size_t>(s) >= D.wide_off.size()) {
        D.wide_off.resize(b.len.size(), -1);
        D.wide_cap.resize(b.len.size(), 0);
        D.packed_deg.resize(b.len.size(), 0);
    }
    const int32_t old = D.packed_deg[s];
    const bool was_hash = D.wide_cap[s] > kSortedRowMax;
    if (d <= kSortedRowMax) {
        if (D.wide_cap[s] < d) {
            // new slot, whole row
            if (!place_row(D, s, pow2_at_least(d))) return false;
            b.sorted_row(s, tmp);
            Edge* row = D.mirror.data() + D.wide_off[s];
            for (int32_t k = 0; k < d; ++k) row[k] = Edge{tmp[k].first, tmp[k].second};
            note_segment(D, out, D.wide_off[s], 0, d);
        } else {
            Edge* row = D.mirror.data() + D.wide_off[s];
            int64_t lowest = d;                                   // lowest position written
            const int32_t k_new = d - old;
            if (k_new > 0) {
                tmp.clear();
                int32_t x = b.head[s];
                for (int32_t k = 0; k < k_new; ++k, x = b.e_next[x]) tmp.emplace_back(b.e_tok[x], b.e_dst[x]);
                std::sort(tmp.begin(), tmp.end());
                int32_t i = old - 1, j = k_new - 1, w = d - 1;
                while (j >= 0) {
                    if (i >= 0 && row[i].tok > tmp[j].first) row[w--] = row[i--];
                    else { row[w] = Edge{tmp[j].first, tmp[j].second}; --w; --j; }
                }
                lowest = w + 1;
            }
            for (size_t q = 0; q < n_redir; ++q) {
                const int32_t tok = redir[q].second;
                int32_t lo = 0, hi = d;
                while (lo < hi) {
                    const int32_t mid = (lo + hi) >> 1;
                    if (row[mid].tok < tok) lo = mid + 1; else hi = mid;
                }
                if (lo < d && row[lo].tok == tok) {
                    const int32_t e = b.find(s, tok);
                    if (e >= 0) row[lo].dst = b.e_dst[e];
                    if (lo < lowest) lowest = lo;
                }
            }
            note_segment(D, out, D.wide_off[s], lowest, d - lowest);
        }
    } else if (!was_hash || 2 * static_cast<int64_t>(d) > D.wide_cap[s]) {
        // a fresh hash table (the row was a sorted array so far, or the table is half full), sent whole
        const int32_t lc = hash_log2cap(d, 4);
        if (!place_row(D, s, 1 << lc)) return false;
        Edge* row = D.mirror.data() + D.wide_off[s];
        for (int32_t k = 0; k < (1 << lc); ++k) row[k] = Edge{-1, -1};
        for (int32_t x = b.head[s]; x >= 0; x = b.e_next[x]) row[hash_find(row, lc, b.e_tok[x])] = Edge{b.e_tok[x], b.e_dst[x]};
        note_segment(D, out, D.wide_off[s], 0, int64_t(1) << lc);
    } else {
        int32_t lc = 0;
        while ((1 << lc) < D.wide_cap[s]) ++lc;
        Edge* row = D.mirror.data() + D.wide_off[s];
        int32_t x = b.head[s];
        for (int32_t k = 0; k < d - old; ++k, x = b.e_next[x]) {          // the transitions added since the last packing
            const uint32_t at = hash_find(row, lc, b.e_tok[x]);
            row[at] = Edge{b.e_tok[x], b.e_dst[x]};
            note_segment(D, out, D.wide_off[s], at, 1);
        }
        for (size_t q = 0; q < n_redir; ++q) {
            const int32_t tok = redir[q].second;
            const uint32_t at = hash_find(row, lc, tok);
            const int32_t e = b.find(s, tok);
            if (row[at].tok == tok && e >= 0 && row[at].dst != b.e_dst[e]) {
                row[at].dst = b.e_dst[e];
                note_segment(D, out, D.wide_off[s], at, 1);
            }
        }
    }
    D.packed_deg[s] = d;
    r->e[0] = D.wide_off[s];
    if (D.wide_cap[s] > kSortedRowMax) {
        int32_t lc = 0;
        while ((1 << lc) < D.wide_cap[s]) ++lc;
        r->e[1] = lc;
    }
    return true;
}

// Everything, laid out afresh (wide rows compacted).
int pack_full(DynIndex& D, Delta* out) {
    const Builder& b = D.b;
    const int64_t S = static_cast<int64_t>(b.len.size());
    out->full = true;
    out->all_rec.assign(static_cast<size_t>(S), StateRec{});
    out->all_root.assign(static_cast<size_t>(D.span_cap), -1);
    D.wide_off.assign(static_cast<size_t>(S), -1);
    D.wide_cap.assign(static_cast<size_t>(S), 0);
    D.packed_deg.assign(static_cast<size_t>(S), 0);
    D.mirror.clear();
    D.w_used = 0;
    std::vector<std::pair<int32_t, int32_t>> tmp;
    for (int64_t s = 1; s < S; ++s) {
        if (!pack_state(D, static_cast<int32_t>(s), &out->all_rec[s], nullptr, 0, tmp, nullptr)) return SAM_ERR_TOO_LARGE;
    }
    out->all_wide.assign(D.mirror.begin(), D.mirror.begin() + D.w_used);
    StateRec& r0 = out->all_rec[0];
    r0.len = 0; r0.link = -1; r0.firstpos = -1; r0.deg = b.deg[0];
    r0.e[0] = r0.e[1] = r0.e[2] = r0.e[3] = -1;
    for (int32_t x = b.head[0]; x >= 0; x = b.e_next[x]) out->all_root[b.e_tok[x]] = b.e_dst[x];
    out->all_corpus = D.corpus;
    out->n_states_after = S;
    out->n_tokens_after = static_cast<int64_t>(D.corpus.size());
    return SAM_OK;
}

// What the last chunk changed.
int pack_changes(DynIndex& D, int64_t corpus_before, Delta* out) {
    Builder& b = D.b;
    std::vector<std::pair<int32_t, int32_t>> tmp;
    out->rec_ids.reserve(b.dirty.size());
    out->recs.reserve(b.dirty.size());
    std::sort(b.redirected.begin(), b.redirected.end());
    const int64_t every = D.relayout_every.load();
    if (every > 0 && ++D.updates_packed % every == 0) {
        Delta fresh;
        const int rc = pack_full(D, &fresh);
        *out = std::move(fresh);
        return rc;
    }
    std::sort(b.dirty.begin(), b.dirty.end());      // new states are consecutive: mostly sequential memory from here on
    for (int32_t s : b.dirty) {
        StateRec r;
        auto lo = b.redirected.end(), hi = b.redirected.end();
        if (b.deg[s] >= 3) {                         // inline records are rebuilt from the chain; only rows need the list
            lo = std::lower_bound(b.redirected.begin(), b.redirected.end(), std::make_pair(s, INT32_MIN));
            hi = std::lower_bound(lo, b.redirected.end(), std::make_pair(s + 1, INT32_MIN));
        }
        if (!pack_state(D, s, &r, lo == hi ? nullptr : &*lo, static_cast<size_t>(hi - lo), tmp, out)) {
            // wide area exhausted: lay everything out afresh and send the whole image instead
            Delta fresh;
            const int rc = pack_full(D, &fresh);
            *out = std::move(fresh);
            return rc;
        }
        out->rec_ids.push_back(s);
        out->recs.push_back(r);
    }
    // root: the last change of a token wins
    std::unordered_map<int32_t, int32_t> last;
    last.reserve(b.root_changes.size() * 2 + 1);
    for (const auto& c : b.root_changes) last[c.first] = c.second;
    out->root_tok.reserve(last.size());
    out->root_dst.reserve(last.size());
    for (const auto& kv : last) { out->root_tok.push_back(kv.first); out->root_dst.push_back(kv.second); }
    out->corpus_off = corpus_before;
    out->corpus_tail.assign(D.corpus.begin() + corpus_before, D.corpus.end());
    out->n_states_after = static_cast<int64_t>(b.len.size());
    out->n_tokens_after = static_cast<int64_t>(D.corpus.size());
    return SAM_OK;
}

void worker_main(DynIndex* D) {
    for (;;) {
        std::vector<int32_t> chunk;
        {
            std::unique_lock<std::mutex> lk(D->mu);
            D->cv_work.wait(lk, [&] { return D->stop || !D->inbox.empty(); });
            if (D->stop) return;
            chunk.swap(D->inbox.front());
            D->inbox.pop_front();
            D->busy = true;
        }
        Delta delta;
        int rc = SAM_OK;
        try {
            const int64_t before = static_cast<int64_t>(D->corpus.size());
            for (int32_t c : chunk) {
                D->b.extend(c, static_cast<int32_t>(D->corpus.size()), D->last);
                D->corpus.push_back(c);
            }
            rc = pack_changes(*D, before, &delta);
            D->b.clear_changes();
        } catch (const std::bad_alloc&) {
            rc = SAM_ERR_NOMEM;
        }
        delta.status = rc;
        if (rc == SAM_OK && D->owner) ring_stage_async(D->owner, &delta);   // on its way to the device before anyone asks
        {
            std::lock_guard<std::mutex> lk(D->mu);
            if (rc != SAM_OK) D->error = rc;
            D->built += static_cast<int64_t>(chunk.size());
            D->ready.push_back(std::move(delta));
            D->busy = false;
        }
        D->cv_idle.notify_all();
    }
}

}  // namespace

int dyn_create(sam_index* idx, const int32_t* corpus, int64_t n, int64_t max_tokens, int32_t max_token_id) {
    if (max_tokens < n || max_tokens < 1 || max_tokens > (int64_t(1) << 29) || max_token_id < 0 ||
        max_token_id >= (1 << 24))
        return SAM_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i)
        if (corpus[i] > max_token_id) return SAM_ERR_INVALID_ARG;
    DynIndex* D = nullptr;
    try {
        D = new DynIndex();
        D->owner = idx;
        D->max_tokens = max_tokens;
        D->s_cap = 2 * max_tokens + 2;
        // sorted rows sit in power-of-two slots (less than twice their length), hash rows are between an eighth
        // and a half full; 8 edges of room per token leaves ample slack for the corpora this is meant for, and
        // when the area does fill up the rows are laid out afresh (SAM_ERR_TOO_LARGE if even that does not fit)
        D->w_cap = std::min<int64_t>(8 * max_tokens + 1024, (int64_t(1) << 31) - 64);
        D->span_cap = static_cast<int64_t>(max_token_id) + 1;
        Builder& b = D->b;
        b.hash_alloc(1u << 16);
        b.new_state(0, -1, -1);
        D->corpus.reserve(static_cast<size_t>(std::min<int64_t>(max_tokens, n + (int64_t(1) << 20))));
        for (int64_t i = 0; i < n; ++i) {
            b.extend(corpus[i], static_cast<int32_t>(i), D->last);
            D->corpus.push_back(corpus[i]);
        }
        b.track = true;
        b.mark.assign(b.len.size(), 0);
        D->queued = D->built = n;
    } catch (const std::bad_alloc&) {
        delete D;
        return SAM_ERR_NOMEM;
    }
    auto up = [](int64_t x) { return (x + 255) & ~int64_t(255); };
    DeviceLayout& L = idx->layout;
    L.n_states = static_cast<int64_t>(D->b.len.size());
    L.n_corpus = n;
    L.root_span = D->span_cap;
    L.n_wide_edges = D->w_cap;
    L.stage_bytes = int64_t(8) << 20;
    L.rec_off = 0;
    L.edge_off = up(L.rec_off + D->s_cap * static_cast<int64_t>(sizeof(StateRec)));
    L.root_off = up(L.edge_off + D->w_cap * static_cast<int64_t>(sizeof(Edge)));
    L.corpus_off = up(L.root_off + D->span_cap * 4);
    L.stage_off = up(L.corpus_off + max_tokens * 4);
    L.ring_off = up(L.stage_off + L.stage_bytes);
    L.ctrl_off = up(L.ring_off + kRingSlots * kRingSlotBytes);
    L.total = up(L.ctrl_off + 256);
    idx->dyn = D;
    D->worker = std::thread(worker_main, D);
    return SAM_OK;
}

void dyn_destroy(sam_index* idx) {
    DynIndex* D = idx->dyn;
    if (!D) return;
    {
        std::lock_guard<std::mutex> lk(D->mu);
        D->stop = true;
    }
    D->cv_work.notify_all();
    if (D->worker.joinable()) D->worker.join();
    delete D;
    idx->dyn = nullptr;
}

int dyn_enqueue(sam_index* idx, const int32_t* tokens, int64_t n) {
    DynIndex* D = idx->dyn;
    if (!D || n < 0 || (n > 0 && !tokens)) return SAM_ERR_INVALID_ARG;
    if (n == 0) return SAM_OK;
    for (int64_t i = 0; i < n; ++i)
        if (tokens[i] < 0 || tokens[i] >= D->span_cap) return SAM_ERR_INVALID_ARG;
    {
        std::lock_guard<std::mutex> lk(D->mu);
        if (D->error != SAM_OK) return D->error;
        if (D->queued + n > D->max_tokens) return SAM_ERR_TOO_LARGE;
        try {
            D->inbox.emplace_back(tokens, tokens + n);
        } catch (const std::bad_alloc&) {
            return SAM_ERR_NOMEM;
        }
        D->queued += n;
    }
    D->cv_work.notify_one();
    return SAM_OK;
}

int dyn_wait(sam_index* idx) {
    DynIndex* D = idx->dyn;
    if (!D) return SAM_ERR_INVALID_ARG;
    std::unique_lock<std::mutex> lk(D->mu);
    D->cv_idle.wait(lk, [&] { return D->inbox.empty() && !D->busy; });
    return D->error;
}

bool dyn_pop_ready(sam_index* idx, Delta* out) {
    DynIndex* D = idx->dyn;
    std::lock_guard<std::mutex> lk(D->mu);
    if (D->ready.empty()) return false;
    *out = std::move(D->ready.front());
    D->ready.pop_front();
    return true;
}

int dyn_full_image(sam_index* idx, Delta* out) {
    DynIndex* D = idx->dyn;
    if (!D) return SAM_ERR_INVALID_ARG;
    std::unique_lock<std::mutex> lk(D->mu);
    D->cv_idle.wait(lk, [&] { return D->inbox.empty() && !D->busy; });
    D->ready.clear();            // whatever they held is part of the image
    try {
        return pack_full(*D, out);
    } catch (const std::bad_alloc&) {
        return SAM_ERR_NOMEM;
    }
}

int dyn_refresh_csr(sam_index* idx) {
    DynIndex* D = idx->dyn;
    if (!D) return SAM_ERR_INVALID_ARG;
    std::unique_lock<std::mutex> lk(D->mu);
    D->cv_idle.wait(lk, [&] { return D->inbox.empty() && !D->busy; });
    try {
        const Builder& b = D->b;
        const size_t S = b.len.size(), E = b.e_tok.size();
        idx->len = b.len;
        idx->link = b.link;
        idx->firstpos = b.fpos;
        idx->row_ptr.resize(S + 1);
        idx->edge_tok.resize(E);
        idx->edge_dst.resize(E);
        std::vector<std::pair<int32_t, int32_t>> row;
        int64_t off = 0;
        for (size_t s = 0; s < S; ++s) {
            idx->row_ptr[s] = off;
            b.sorted_row(static_cast<int32_t>(s), row);
            for (const auto& e : row) {
                idx->edge_tok[off] = e.first;
                idx->edge_dst[off] = e.second;
                ++off;
            }
        }
        idx->row_ptr[S] = off;
        idx->layout.n_states = static_cast<int64_t>(S);
    } catch (const std::bad_alloc&) {
        return SAM_ERR_NOMEM;
    }
    return SAM_OK;
}

int dyn_sizes(sam_index* idx, int64_t* n_states, int64_t* n_edges) {
    DynIndex* D = idx->dyn;
    if (!D) return SAM_ERR_INVALID_ARG;
    std::unique_lock<std::mutex> lk(D->mu);
    D->cv_idle.wait(lk, [&] { return D->inbox.empty() && !D->busy; });
    if (n_states) *n_states = static_cast<int64_t>(D->b.len.size());
    if (n_edges) *n_edges = static_cast<int64_t>(D->b.e_tok.size());
    return SAM_OK;
}

void staged_layout(const Delta& D, StagedLayout* out) {
    auto up32 = [](int64_t x) { return (x + 31) & ~int64_t(31); };
    int64_t n_seg = 0, n_edges = 0;
    for (const WideSeg& g : D.segs)
        if (g.len < kDirectRowEdges) { ++n_seg; n_edges += g.len; }
    const int64_t n_rec = static_cast<int64_t>(D.rec_ids.size());
    const int64_t n_root = static_cast<int64_t>(D.root_tok.size());
    const int64_t n_tail = static_cast<int64_t>(D.corpus_tail.size());
    StagedLayout& a = *out;
    a.off_ids = 0;
    a.off_recs = up32(n_rec * 4);
    a.off_descs = a.off_recs + n_rec * static_cast<int64_t>(sizeof(StateRec));
    a.off_edges = up32(a.off_descs + n_seg * 16);
    a.off_rtok = up32(a.off_edges + n_edges * static_cast<int64_t>(sizeof(Edge)));
    a.off_rdst = up32(a.off_rtok + n_root * 4);
    a.off_tail = up32(a.off_rdst + n_root * 4);
    a.total = up32(a.off_tail + n_tail * 4);
    a.n_rec = static_cast<int32_t>(n_rec);
    a.n_seg = static_cast<int32_t>(n_seg);
    a.n_root = static_cast<int32_t>(n_root);
    a.n_tail = static_cast<int32_t>(n_tail);
}

void staged_fill(const Delta& D, const StagedLayout& a, char* h) {
    // row descriptor as the device reads it: {int64 first edge in the wide array, int32 first edge in the list, int32 length}
    struct Desc { long long dst_off; int src_off; int len; };
    static_assert(sizeof(Desc) == 16, "row descriptor");
    std::memcpy(h + a.off_ids, D.rec_ids.data(), static_cast<size_t>(a.n_rec) * 4);
    std::memcpy(h + a.off_recs, D.recs.data(), static_cast<size_t>(a.n_rec) * sizeof(StateRec));
    Desc* descs = reinterpret_cast<Desc*>(h + a.off_descs);
    Edge* edges = reinterpret_cast<Edge*>(h + a.off_edges);
    int64_t ns = 0, ne = 0;
    for (const WideSeg& g : D.segs) {
        if (g.len >= kDirectRowEdges) continue;
        descs[ns++] = Desc{g.dst_off, static_cast<int>(ne), g.len};
        std::memcpy(edges + ne, D.seg_edges.data() + g.src_off, static_cast<size_t>(g.len) * sizeof(Edge));
        ne += g.len;
    }
    std::memcpy(h + a.off_rtok, D.root_tok.data(), static_cast<size_t>(a.n_root) * 4);
    std::memcpy(h + a.off_rdst, D.root_dst.data(), static_cast<size_t>(a.n_root) * 4);
    std::memcpy(h + a.off_tail, D.corpus_tail.data(), static_cast<size_t>(a.n_tail) * 4);
}

int dyn_set_relayout_every(sam_index* idx, int64_t every) {
    DynIndex* D = idx->dyn;
    if (!D || every < 0) return SAM_ERR_INVALID_ARG;
    D->relayout_every.store(every);
    return SAM_OK;
}

void dyn_counts(sam_index* idx, int64_t* queued, int64_t* built) {
    DynIndex* D = idx->dyn;
    std::lock_guard<std::mutex> lk(D->mu);
    if (queued) *queued = D->queued;
    if (built) *built = D->built;
}

}  // namespace samb200
