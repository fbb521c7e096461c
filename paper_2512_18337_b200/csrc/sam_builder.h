// Internal: the online suffix-automaton builder shared by the one-shot build and the growing index.
//
// Container strategy: every transition is a node of one global pool, chained per source
// state (newest first).  States with few transitions are searched by walking their chain;
// once a state has more than kHeavy transitions all of them are also indexed in one
// open-addressing hash table keyed by (state, token).  Rows are sorted by token id only
// when they are exported or packed for the device.
//
// With `track` set the builder also records which states changed (new state, new or redirected
// transition, new suffix link) and which root transitions changed, so that a growing index can
// send the device only what differs.
#pragma once
#include <algorithm>
#include <cstdint>
#include <utility>
#include <vector>

namespace samb200 {

constexpr int32_t kHeavy = 6;
constexpr uint64_t kEmptyKey = ~0ull;

struct Builder {
    std::vector<int32_t> len, link, fpos, head, deg;
    std::vector<int32_t> e_tok, e_dst, e_next;
    std::vector<uint64_t> hkey;
    std::vector<int32_t> hval;
    uint64_t hmask = 0;
    int64_t hcount = 0;

    bool track = false;
    std::vector<uint8_t> mark;                              // state already in `dirty`
    std::vector<int32_t> dirty;                             // non-root states to repack
    std::vector<std::pair<int32_t, int32_t>> root_changes;  // (token, destination) in order of change
    std::vector<std::pair<int32_t, int32_t>> redirected;    // (state, token) of transitions that got a new destination

    void touch(int32_t s) {
        if (!track || s == 0) return;
        if (!mark[s]) { mark[s] = 1; dirty.push_back(s); }
    }
    void clear_changes() {
        for (int32_t s : dirty) mark[s] = 0;
        dirty.clear();
        root_changes.clear();
        redirected.clear();
    }

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
        hkey.assign(size, kEmptyKey);
        hval.assign(size, -1);
        hmask = size - 1;
    }
    void hash_put_raw(uint64_t k, int32_t e) {
        uint64_t i = mix(k) & hmask;
        while (hkey[i] != kEmptyKey) i = (i + 1) & hmask;
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
                if (ok[i] != kEmptyKey) hash_put_raw(ok[i], ov[i]);
        }
        hash_put_raw(key_of(s, c), e);
        ++hcount;
    }
    int32_t hash_get(int32_t s, int32_t c) const {
        const uint64_t k = key_of(s, c);
        uint64_t i = mix(k) & hmask;
        while (hkey[i] != kEmptyKey) {
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
        if (track) mark.push_back(0);
        const int32_t id = static_cast<int32_t>(len.size() - 1);
        touch(id);
        return id;
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
        touch(s);
        if (track && s == 0) root_changes.emplace_back(c, d);
    }

    // One step of the online construction: append token c at text position pos.
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
                    touch(p);
                    if (track && p == 0) root_changes.emplace_back(c, clone);
                    if (track && p != 0) redirected.emplace_back(p, c);
                    p = link[p];
                }
                link[q] = clone;
                touch(q);
                link[cur] = clone;
            }
        }
        last = cur;
    }

    // Transitions of state s, ascending by token.
    void sorted_row(int32_t s, std::vector<std::pair<int32_t, int32_t>>& out) const {
        out.clear();
        for (int32_t x = head[s]; x >= 0; x = e_next[x]) out.emplace_back(e_tok[x], e_dst[x]);
        std::sort(out.begin(), out.end());
    }
};

}  // namespace samb200
