// Device code of the draft + verify path (sm_100a). Included only by sam_capi.cu.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "sam_index.h"

namespace samb200 {

constexpr unsigned kFull = 0xFFFFFFFFu;

// ============================================================================================
// Automaton walk and draft emission (Section 5.4.2; Algorithm 3 "FollowTransitions" / "Emit").
// One warp per request stream; every lane holds the same (state, matched_len, record).
// ============================================================================================

struct RecRegs {
    int4 a;  // len, link, firstpos, deg
    int4 b;  // inline transitions / wide-row offset
};

__device__ __forceinline__ RecRegs load_rec(const DeviceSam& sam, int s) {
    const int4* p = reinterpret_cast<const int4*>(sam.rec + s);
    RecRegs r;
    r.a = __ldg(p);
    r.b = __ldg(p + 1);
    return r;
}

__device__ __forceinline__ RecRegs root_rec() {
    RecRegs r;
    r.a = make_int4(0, -1, -1, 0);
    r.b = make_int4(-1, -1, -1, -1);
    return r;
}

// One warp-wide read of an ascending row of at most 32 (tok, dst) pairs.
__device__ __forceinline__ int sorted_row_lookup(const Edge* __restrict__ row, int deg, int c, int lane) {
    int2 e = make_int2(0, -1);
    const bool in = lane < deg;
    if (in) e = __ldg(reinterpret_cast<const int2*>(row + lane));
    const unsigned hit = __ballot_sync(kFull, in && e.x == c);
    if (hit == 0) return -1;
    return __shfl_sync(kFull, e.y, __ffs(hit) - 1);
}

// Hash row: 32 consecutive slots from the token's home slot per round.  Insertion took the first empty
// slot from there and nothing is ever deleted, so a token that is present sits before the first empty slot.
__device__ __forceinline__ int hash_row_lookup(const Edge* __restrict__ row, int log2cap, int c, int lane) {
    if (c < 0) return -1;
    const unsigned mask = (1u << log2cap) - 1u;
    const unsigned home = hash_slot(c, log2cap);
    for (unsigned w = 0; w <= mask; w += 32) {
        const int2 e = __ldg(reinterpret_cast<const int2*>(row + ((home + w + lane) & mask)));
        const unsigned hit = __ballot_sync(kFull, e.x == c);
        if (hit != 0) return __shfl_sync(kFull, e.y, __ffs(hit) - 1);
        if (__ballot_sync(kFull, e.x < 0) != 0) return -1;
    }
    return -1;
}

// Destination of the transition (s, c) or -1. `r` is the record of s.
__device__ __forceinline__ int transition(const DeviceSam& sam, int s, const RecRegs& r, int c, int lane) {
    if (s == 0) {
        return (c >= 0 && c < sam.root_span) ? __ldg(sam.root_dst + c) : -1;
    }
    const int deg = r.a.w;
    if (deg <= 2) {
        if (deg >= 1 && r.b.x == c) return r.b.y;
        if (deg == 2 && r.b.z == c) return r.b.w;
        return -1;
    }
    if (deg <= kSortedRowMax) return sorted_row_lookup(sam.wide + r.b.x, deg, c, lane);
    return hash_row_lookup(sam.wide + r.b.x, r.b.y, c, lane);
}

// Consume one token: a transition extends the match by one; on a miss follow the suffix link
// and shorten the match to that state's length; a miss at the root resets the match to zero.
__device__ __forceinline__ void walk_token(const DeviceSam& sam, int c, int& s, int& L, RecRegs& r, int lane) {
    for (;;) {
        const int d = transition(sam, s, r, c, lane);
        if (d >= 0) {
            s = d;
            L += 1;
            r = load_rec(sam, s);
            return;
        }
        if (s == 0) {
            L = 0;
            return;
        }
        s = r.a.y;
        r = (s == 0) ? root_rec() : load_rec(sam, s);
        L = r.a.x;
    }
}

// A (state, matched_len) pair that this library did not produce is reset to the start pair
// instead of being dereferenced.
__device__ __forceinline__ void sanitize_stream_state(const DeviceSam& sam, int& s, int& L) {
    if (s <= 0 || s >= sam.n_states || L < 0) {
        s = 0;
        L = 0;
    }
}

__device__ __forceinline__ bool is_separator(const DeviceSam& sam, int tok) {
    bool hit = false;
#pragma unroll 1
    for (int k = 0; k < sam.n_sep; ++k) hit |= (sam.seps[k] == tok);
    return hit;
}

// Emit the continuation after the first occurrence of the matched suffix (K <= 32: one lane
// per draft slot, one coalesced read of the corpus). Returns n_draft (same on every lane).
__device__ __forceinline__ int emit_draft(const DeviceSam& sam, int L, const RecRegs& r, int K, int min_match,
                                          int* __restrict__ drafts_row, int lane) {
    int nd = 0;
    int tok = -1;
    if (L >= min_match) {                     // uniform across the warp
        const int64_t pos = static_cast<int64_t>(r.a.z) + 1 + lane;
        bool stop = true;
        if (lane < K && pos < sam.n_corpus) {
            tok = __ldg(sam.corpus + pos);
            stop = is_separator(sam, tok);
        }
        const unsigned sm = __ballot_sync(kFull, stop);   // lanes >= K always stop
        nd = __ffs(sm) - 1;                   // sm != 0 because K <= 32 and lane K.. stop (or nd = K)
        if (sm == 0) nd = K;                  // K == 32 and nothing stopped
        nd = min(nd, K);
    }
    if (lane < K) drafts_row[lane] = (lane < nd) ? tok : -1;
    return nd;
}

// sam_draft: walk caller-provided tokens, then emit.
__global__ void __launch_bounds__(128)
draft_kernel(DeviceSam sam, int B, int* __restrict__ state, int* __restrict__ matched_len,
             const int* __restrict__ new_tokens, int ld, const int* __restrict__ n_new,
             int K, int min_match, int* __restrict__ drafts, int* __restrict__ n_draft) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (b >= B) return;
    int s = state[b];
    int L = matched_len[b];
    sanitize_stream_state(sam, s, L);
    RecRegs r = (s == 0) ? root_rec() : load_rec(sam, s);
    const int n = max(0, min(n_new[b], ld));
    const int* row = new_tokens + static_cast<int64_t>(b) * ld;
    for (int base = 0; base < n; base += 32) {
        const int mine = (base + lane < n) ? __ldg(row + base + lane) : -1;
        const int cnt = min(32, n - base);
        for (int t = 0; t < cnt; ++t) {
            const int c = __shfl_sync(kFull, mine, t);
            walk_token(sam, c, s, L, r, lane);
        }
    }
    const int nd = emit_draft(sam, L, r, K, min_match, drafts + static_cast<int64_t>(b) * K, lane);
    if (lane == 0) {
        state[b] = s;
        matched_len[b] = L;
        n_draft[b] = nd;
    }
}

// Composite drafting over several automata (Section 5.4.2: the session's context plus the retrieved
// contexts, weighted by similarity).  One CTA per stream, one warp per slot: every slot follows the
// new tokens in its own automaton from its own (state, matched_len); the draft comes from the slot
// with the largest weight * matched_len (float32) among those that reach min_match, the lowest slot
// winning ties.
constexpr int kMaxSlots = 8;

__global__ void __launch_bounds__(32 * kMaxSlots)
multi_draft_kernel(const DeviceSam* __restrict__ table, int n_members, int B, int M,
                   const int* __restrict__ slots, const float* __restrict__ weights,
                   int* __restrict__ state, int* __restrict__ matched_len,
                   const int* __restrict__ new_tokens, int ld, const int* __restrict__ n_new,
                   int K, int min_match, int* __restrict__ drafts, int* __restrict__ n_draft,
                   int* __restrict__ chosen) {
    __shared__ float score[kMaxSlots];
    __shared__ int ok[kMaxSlots];
    __shared__ int winner;
    const int b = blockIdx.x;
    const int m = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long at = static_cast<long long>(b) * M + m;
    const int member = slots[at];
    const bool live = member >= 0 && member < n_members;
    int s = 0, L = 0;
    RecRegs r = root_rec();
    DeviceSam sam;
    if (live) {
        sam = table[member];
        s = state[at];
        L = matched_len[at];
        sanitize_stream_state(sam, s, L);
        if (s != 0) r = load_rec(sam, s);
        const int n = max(0, min(n_new[b], ld));
        const int* row = new_tokens + static_cast<long long>(b) * ld;
        for (int base = 0; base < n; base += 32) {
            const int mine = (base + lane < n) ? __ldg(row + base + lane) : -1;
            const int cnt = min(32, n - base);
            for (int t = 0; t < cnt; ++t) walk_token(sam, __shfl_sync(kFull, mine, t), s, L, r, lane);
        }
        if (lane == 0) {
            state[at] = s;
            matched_len[at] = L;
        }
    }
    if (lane == 0) {
        ok[m] = live && L >= min_match;
        score[m] = live ? weights[at] * static_cast<float>(L) : 0.0f;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int w = -1;
        float best = 0.0f;
        for (int q = 0; q < M; ++q)
            if (ok[q] && (w < 0 || score[q] > best)) { w = q; best = score[q]; }
        winner = w;
        chosen[b] = w;
        if (w < 0) n_draft[b] = 0;
    }
    __syncthreads();
    if (winner == m) {
        const int nd = emit_draft(sam, L, r, K, min_match, drafts + static_cast<long long>(b) * K, lane);
        if (lane == 0) n_draft[b] = nd;
    } else if (winner < 0 && m == 0 && lane < K) {
        drafts[static_cast<long long>(b) * K + lane] = -1;
    }
}

// Composite step after the argmax: warp 0 accepts (decode, longest matching prefix, the model's own token),
// then every slot resumes from the state its walk-ahead reached after the accepted prefix, follows the model's
// token in its own automaton, and the slots compete for the next draft as in multi_draft_kernel.
// Declared here, defined after accept_stream.
struct AcceptArgs;
struct MultiArgs {
    const DeviceSam* table;
    int n_members, M;
    const int* slots;          // [B, M]
    const float* weights;      // [B, M]
    int* state;                // [B, M]
    int* matched_len;          // [B, M]
    const int* pre_state;      // [B, M, K]
    const int* pre_len;        // [B, M, K]
    int* chosen;               // [B]
};

// Walk-ahead along the draft.  While the logits of a step are still being reduced, spare warps
// follow the automaton over each stream's DRAFT tokens and record the (state, matched_len)
// reached after every prefix.  Whatever prefix the verification later accepts, the walk over it
// is then already done and only the model's own token remains to be followed.
struct PreWalk {
    const int* state;        // [B] stream state at the start of the step
    const int* matched_len;  // [B]
    const int* drafts;       // [B, K]
    const int* n_draft;      // [B]
    int* pre_state;          // [B, K] state after drafts[b, 0..j]
    int* pre_len;            // [B, K] matched_len after drafts[b, 0..j]
    int B, K;
    int enabled;
    int no_spec;             // speculation is off for this step: every proposal counts as empty
    // composite drafting: M > 0 slots per stream, each with its own automaton and state;
    // state / matched_len / pre_state / pre_len are then indexed by b * M + m
    const DeviceSam* table;
    const int* slots;        // [B, M] member number or -1
    int M, n_members;
};

// `at` indexes the state arrays (b for a single automaton, b * M + m for a slot); the drafts are stream b's.
__device__ __forceinline__ void prewalk_stream(const DeviceSam& sam, const PreWalk& pw, int b, int at, int lane) {
    int s = pw.state[at];
    int L = pw.matched_len[at];
    sanitize_stream_state(sam, s, L);
    const int nd = pw.no_spec ? 0 : max(0, min(pw.n_draft[b], pw.K));
    const int d = (lane < nd) ? pw.drafts[static_cast<long long>(b) * pw.K + lane] : -1;
    if (nd == 0) return;
    RecRegs r = (s == 0) ? root_rec() : load_rec(sam, s);
    int my_s = 0, my_L = 0;
    for (int j = 0; j < nd; ++j) {
        const int c = __shfl_sync(kFull, d, j);
        walk_token(sam, c, s, L, r, lane);
        if (lane == j) { my_s = s; my_L = L; }
    }
    if (lane < nd) {
        pw.pre_state[static_cast<long long>(at) * pw.K + lane] = my_s;
        pw.pre_len[static_cast<long long>(at) * pw.K + lane] = my_L;
    }
}

// ============================================================================================
// Vocabulary argmax (Algorithm 3 "Validate with main LLM": the model's greedy choice per row).
// Bandwidth-bound: every bf16 is read once. Ties go to the lowest index.
// ============================================================================================

// Monotone 16-bit key of a non-NaN bf16 value held in a float; -0 and +0 share a key; >= 1.
__device__ __forceinline__ unsigned ordered_key(float x) {
    unsigned b = __float_as_uint(x) >> 16;
    if ((b & 0x7FFFu) == 0) b = 0;
    return (b & 0x8000u) ? (~b & 0xFFFFu) : (b | 0x8000u);
}

// (value key, index) packed so that an unsigned 64-bit max picks the larger value and,
// among equal values, the smaller index. Zero means "no candidate".
__device__ __forceinline__ unsigned long long pack_candidate(float x, unsigned idx) {
    return (static_cast<unsigned long long>(ordered_key(x)) << 32) | (0xFFFFFFFFu - idx);
}

// A row whose element 0 is NaN keeps index 0 (nothing ever compares greater than NaN): this
// candidate beats every real one (value keys stop at 0xFF80) and decodes to index 0.
constexpr unsigned long long kCandidateFirstIsNaN = 0x0000FFFFFFFFFFFFull;

__device__ __forceinline__ bool bf16_bits_nan(unsigned b) { return (b & 0x7FFFu) > 0x7F80u; }

__device__ __forceinline__ float bf16lo(unsigned u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(unsigned u) { return __uint_as_float(u & 0xFFFF0000u); }

__device__ __forceinline__ unsigned hmax2u(unsigned a, unsigned b) {
    __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&a);
    __nv_bfloat162 y = *reinterpret_cast<__nv_bfloat162*>(&b);
    __nv_bfloat162 m = __hmax2(x, y);        // a NaN operand is dropped, as in the scalar scan
    return *reinterpret_cast<unsigned*>(&m);
}

// Maximum of the eight bf16 values of a 16-byte vector (NaN only if all eight are NaN).
__device__ __forceinline__ float vec_max(const uint4& v) {
    const unsigned m = hmax2u(hmax2u(v.x, v.y), hmax2u(v.z, v.w));
    return fmaxf(bf16lo(m), bf16hi(m));
}

constexpr unsigned kNaN2 = 0x7FC07FC0u;

// Replace the lanes of vector q that fall outside virtual elements [off, off + V) by NaN.
__device__ __forceinline__ void mask_vector(uint4& v, long long q, int off, int V) {
    unsigned w[4] = {v.x, v.y, v.z, v.w};
    const long long e0 = q * 8;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const long long lo = e0 + 2 * k, hi = lo + 1;
        if (lo < off || lo >= static_cast<long long>(off) + V) w[k] = (w[k] & 0xFFFF0000u) | 0x7FC0u;
        if (hi < off || hi >= static_cast<long long>(off) + V) w[k] = (w[k] & 0x0000FFFFu) | 0x7FC00000u;
    }
    v = make_uint4(w[0], w[1], w[2], w[3]);
}

// First position (0..7) in the vector whose value equals x; 8 if none.
__device__ __forceinline__ int first_equal(const uint4& v, float x) {
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
    int e = 8;
#pragma unroll
    for (int k = 3; k >= 0; --k) {
        if (bf16hi(w[k]) == x) e = 2 * k + 1;
        if (bf16lo(w[k]) == x) e = 2 * k;
    }
    return e;
}

struct RowView {
    const uint4* vec;   // 16-byte aligned start at or before the row's first element
    int off;            // elements between vec and the row start (0..7)
    int nvec;           // vectors covering the row
};

__device__ __forceinline__ RowView row_view(const __nv_bfloat16* logits, long long stride, long long row, int V) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(logits + row * stride);
    const uintptr_t a0 = a & ~static_cast<uintptr_t>(15);
    RowView rv;
    rv.vec = reinterpret_cast<const uint4*>(a0);
    rv.off = static_cast<int>((a - a0) >> 1);
    rv.nvec = (rv.off + V + 7) >> 3;
    return rv;
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Status word of the verification scratch (sam_workspace_status).
enum : int { kStatusOk = 0, kStatusWaitTimeout = 1, kStatusQueueOverflow = 2, kStatusBadRowList = 3 };

// Optional indirection and offset for the argmax kernels.
//   list / meta:   only the rows list[0..meta[kListCount]) are reduced, in that order (both in device memory);
//                  the list counts only if meta[kListSig] == sig (it was made for this batch shape), otherwise
//                  nothing is reduced and *status is raised.  list == nullptr: all rows 0..R-1.
//   v_offset:      added to every index (the logits are columns v_offset.. of a wider vocabulary).
// meta words: [kListCount] rows in the list; [kListSig] the shape the list was made for; [kListAccum], 8-byte aligned,
// a 64-bit word zero between calls: rows collected so far for the NEXT list (low half) and streams that have added
// theirs (high half).
enum : int { kListCount = 0, kListSig = 1, kListAccum = 2 };
struct RowMap {
    const int* list;
    const int* meta;
    int v_offset;
    int sig;
    int* status;
};
__host__ __device__ __forceinline__ int row_list_sig(int B, int K) {
    return static_cast<int>((static_cast<unsigned>(B) << 6) ^ static_cast<unsigned>(K) ^ 0x5A000000u);
}
// Rows the list holds for this call (0 and a raised status word when the list is not one for this call).
__device__ __forceinline__ long long listed_rows(const RowMap& rm, long long R) {
    const long long n = __ldg(rm.meta + kListCount);
    if (__ldg(rm.meta + kListSig) != rm.sig || n < 0 || n > R) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicExch(rm.status, kStatusBadRowList);
        return 0;
    }
    return n;
}

// Step options (same values as SAM_STEP_* in sam.h).
constexpr unsigned kNoSpeculation = 1u, kSkipUnusedRows = 2u, kRowListReady = 4u;
// Internal: the accept step runs inside the argmax kernel as soon as rows 0 .. n_draft are complete; the rows behind the
// proposal are not its business then (the finisher of the argmax kernel reports them when they are complete).
constexpr unsigned kLeaveUnusedRows = 0x100u;

// Rows 0..n_draft[b] of every stream, in stream order (n_draft clamped to 0..K, or 0 when speculation
// is off); one CTA, a block-wide running sum.  meta receives the count and the shape signature.
__global__ void __launch_bounds__(1024)
build_row_list_kernel(const int* __restrict__ n_draft, int B, int K, unsigned flags,
                      int* __restrict__ list, int* __restrict__ meta) {
    __shared__ int warp_sum[32];
    __shared__ int carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < B; base += blockDim.x) {
        const int b = base + threadIdx.x;
        int need = 0;
        if (b < B) need = ((flags & kNoSpeculation) ? 0 : max(0, min(n_draft[b], K))) + 1;
        int incl = need;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(kFull, incl, d);
            if (lane >= d) incl += o;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        int before = carry;
        for (int w = 0; w < warp; ++w) before += warp_sum[w];
        const int start = before + incl - need;
        for (int j = 0; j < need; ++j) list[start + j] = b * (K + 1) + j;
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry = before + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        meta[kListCount] = carry;
        meta[kListSig] = row_list_sig(B, K);
    }
}

constexpr int kArgmaxThreads = 256;
constexpr int kTileVec = 1024;    // 16-byte vectors per tile: 16 KB
constexpr int kVecPerThread = kTileVec / kArgmaxThreads;

// Turn a thread's (best value, vector index) into a packed candidate by re-reading that one
// vector and locating the first equal element.
__device__ __forceinline__ unsigned long long resolve_candidate(const RowView& rv, int V, float best, int bestq,
                                                                int v_offset) {
    if (bestq < 0) return 0ull;
    uint4 v = __ldg(rv.vec + bestq);
    if (bestq == 0 || bestq == rv.nvec - 1) mask_vector(v, bestq, rv.off, V);
    const int e = first_equal(v, best);
    const unsigned idx = static_cast<unsigned>(bestq * 8 + e - rv.off + v_offset);
    return pack_candidate(best, idx);
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long k) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const unsigned long long o = __shfl_xor_sync(kFull, k, d);
        k = (o > k) ? o : k;
    }
    return k;
}

// Generic streaming argmax: direct 16-byte global loads, any row alignment.
// The R * tiles_per_row tiles are split into equal contiguous ranges, one per CTA; partial
// results of a row meet in keys[row] through a 64-bit atomic max.
// kDirectCtasPerSm CTAs stay resident per SM (the register bound makes room for them): 6 x 16 KB of loads
// in flight per SM measured fastest (4: 205 us, 5: 197 us, 6: 193 us, 7: 195 us, 8: 212 us on one launch of config 2).
constexpr int kDirectCtasPerSm = 6;
__global__ void __launch_bounds__(kArgmaxThreads, kDirectCtasPerSm)
argmax_direct_kernel(const __nv_bfloat16* __restrict__ logits, long long stride, long long R, int V,
                     int tiles_per_row, unsigned long long* __restrict__ keys, RowMap rm) {
    // the accept kernel may be scheduled now; it waits for this grid before it reads any result
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long R_all = R;
    if (rm.list != nullptr) R = listed_rows(rm, R_all);
    const long long total = R * tiles_per_row;
    const long long t0 = total * blockIdx.x / gridDim.x;
    const long long t1 = total * (blockIdx.x + 1) / gridDim.x;
    const int lane = threadIdx.x & 31;
    long long cur_row = -1;
    RowView rv{};
    float best = __int_as_float(0xff800000);   // -inf: only strictly greater values become candidates
    int bestq = -1;
    bool first_nan = false;                    // this thread saw a NaN in element 0 of the current row

    auto flush = [&]() {
        if (cur_row < 0) return;
        // Only a lane that holds the warp's largest value can win, so only those lanes go back to memory for
        // the position of their element (usually one lane; every lane doing so re-read 8 % of the logits).
        float wbest = best;                         // never NaN: only values greater than -inf are kept
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) wbest = fmaxf(wbest, __shfl_xor_sync(kFull, wbest, d));
        unsigned long long k = 0ull;
        if (first_nan) k = kCandidateFirstIsNaN;
        else if (best == wbest) k = resolve_candidate(rv, V, best, bestq, rm.v_offset);
        k = warp_max_u64(k);
        if (lane == 0 && k != 0ull) atomicMax(keys + cur_row, k);
    };

    for (long long t = t0; t < t1; ++t) {
        const long long vrow = t / tiles_per_row;
        const int tile = static_cast<int>(t - vrow * tiles_per_row);
        long long row = vrow;
        if (rm.list != nullptr) {              // clamped: a foreign list can give wrong results, never a fault
            row = __ldg(rm.list + vrow);
            row = row < 0 ? 0 : (row >= R_all ? R_all - 1 : row);
        }
        if (row != cur_row) {
            flush();
            cur_row = row;
            rv = row_view(logits, stride, row, V);
            best = __int_as_float(0xff800000);
            bestq = -1;
            first_nan = false;
        }
        const int q0 = tile * kTileVec + threadIdx.x;
        uint4 v[kVecPerThread];
#pragma unroll
        for (int i = 0; i < kVecPerThread; ++i) {
            const int q = q0 + i * kArgmaxThreads;
            v[i] = make_uint4(kNaN2, kNaN2, kNaN2, kNaN2);
            if (q < rv.nvec) v[i] = ld_stream(rv.vec + q);
        }
#pragma unroll
        for (int i = 0; i < kVecPerThread; ++i) {
            const int q = q0 + i * kArgmaxThreads;
            if (q < rv.nvec) {
                if (q == 0) {
                    const int h = rv.off >> 1;
                    const unsigned pair = (h == 0) ? v[i].x : (h == 1) ? v[i].y : (h == 2) ? v[i].z : v[i].w;
                    first_nan = rm.v_offset == 0 && bf16_bits_nan((rv.off & 1) ? (pair >> 16) : (pair & 0xFFFFu));
                }
                if (q == 0 || q == rv.nvec - 1) mask_vector(v[i], q, rv.off, V);
                const float m = vec_max(v[i]);
                if (m > best) { best = m; bestq = q; }
            }
        }
    }
    flush();
}

// ============================================================================================
// Accept + feedback (Algorithm 3: commit the matched prefix, fall back to the model's token at
// the first mismatch, then follow the automaton over what was committed and draft again).
// One warp per stream. Also decodes the packed argmax candidates and re-zeroes them.
// ============================================================================================
enum : int { kTailVerifyOnly = 0, kTailFullWalk = 1, kTailResume = 2 };

// Everything the accept step of one stream reads and writes (device pointers of the caller).
struct AcceptArgs {
    const __nv_bfloat16* logits;
    long long stride;
    int B, K;
    const int* drafts;        // [B, K]
    const int* n_draft;       // [B]
    int* argmax_out;          // [B, K+1]
    int* accepted;            // [B, K+1]
    int* n_accepted;          // [B]
    unsigned long long* keys; // [B*(K+1)] packed argmax candidates, re-zeroed here
    int* state;               // [B] (unused in kTailVerifyOnly)
    int* matched_len;         // [B]
    int min_match;
    int* next_drafts;         // [B, K]
    int* next_n_draft;        // [B]
    const int* pre_state;     // [B, K] walk-ahead results (kTailResume)
    const int* pre_len;       // [B, K]
    unsigned flags;           // kNoSpeculation | kSkipUnusedRows
    unsigned long long* counters;   // [6] running statistics, or nullptr
    int* next_list;           // row list of the NEXT step (rows 0..next_n_draft[b] of every stream, any order), or nullptr
    int* list_meta;           // its meta words (see RowMap)
    int* acc_epoch;           // [B] number of the launch in which the stream's accept step last ran inside the argmax kernel, or nullptr
};

// One warp, one stream.  The packed candidates and the walk-ahead results may have been produced
// by other SMs moments ago, so they are read past L1 (ld.cg).
// kAfterGrid: the kernel was launched as a programmatic dependent of the argmax kernel - everything that
// does not depend on that kernel's output is loaded first, then the warp waits for it to finish.
template <int kMode, bool kAfterGrid = false>
__device__ __forceinline__ void accept_stream(const DeviceSam& sam, const AcceptArgs& p, int b, int lane,
                                              int* out_a = nullptr, int* out_bonus = nullptr, int epoch = 0) {
    const int K = p.K;
    const int K1 = K + 1;
    const long long row0 = static_cast<long long>(b) * K1;
    // independent loads first, so that they travel together
    int ps = 0, pl = 0, s = 0, L = 0;
    RecRegs r = root_rec();
    if (kMode != kTailVerifyOnly) {
        s = p.state[b];
        L = p.matched_len[b];
        sanitize_stream_state(sam, s, L);
        if (s != 0) r = load_rec(sam, s);
    }
    const int nd = (p.flags & kNoSpeculation) ? 0 : max(0, min(p.n_draft[b], K));
    const int d = (lane < K) ? p.drafts[static_cast<long long>(b) * K + lane] : -1;
    RecRegs rj = root_rec();     // lane j: record of the state reached after j + 1 drafts
    // Launched as a dependent of the argmax kernel and with no walk-ahead done there: the time until that grid has
    // finished is used to follow the whole proposal here, lane j keeping what was reached after j + 1 drafts.
    constexpr bool kWalkBeforeWait = kMode == kTailFullWalk && kAfterGrid;
    if (kWalkBeforeWait) {
        int s2 = s, L2 = L;
        RecRegs r2 = r;
        for (int j = 0; j < nd; ++j) {
            walk_token(sam, __shfl_sync(kFull, d, j), s2, L2, r2, lane);
            if (lane == j) { ps = s2; pl = L2; rj = r2; }
        }
    }
    if (kAfterGrid) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (kMode == kTailResume && lane < nd) {
        ps = __ldcg(p.pre_state + static_cast<long long>(b) * K + lane);
        pl = __ldcg(p.pre_len + static_cast<long long>(b) * K + lane);
        // every possible resume point is fetched now, while the row results are still on their way
        if (ps > 0 && ps < sam.n_states) rj = load_rec(sam, ps);
    }

    // rows j = lane and j = lane + 32 (K + 1 <= 33)
    int am[2] = {-1, -1};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int j = lane + 32 * h;
        if (j < K1 && !((p.flags & kLeaveUnusedRows) && j > nd)) {
            const unsigned long long k = __ldcg(p.keys + row0 + j);
            p.keys[row0 + j] = 0ull;
            // no candidate at all (nothing in the row is greater than -inf): index 0, as a scan from element 0 gives
            int idx = (k != 0ull) ? static_cast<int>(0xFFFFFFFFu - static_cast<unsigned>(k)) : 0;
            if ((p.flags & kSkipUnusedRows) && j > nd) idx = -1;        // the row was not looked at
            am[h] = idx;
            p.argmax_out[row0 + j] = idx;
        }
    }

    const unsigned mism = __ballot_sync(kFull, lane < nd && d != am[0]);
    const int a = mism ? (__ffs(mism) - 1) : nd;        // accepted draft tokens
    const int bonus_lo = __shfl_sync(kFull, am[0], a & 31);
    const int bonus_hi = __shfl_sync(kFull, am[1], 0);
    const int bonus = (a < 32) ? bonus_lo : bonus_hi;
    if (out_a) *out_a = a;
    if (out_bonus) *out_bonus = bonus;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int j = lane + 32 * h;
        if (j < K1) p.accepted[row0 + j] = (j < a) ? d : ((j == a) ? bonus : -1);
    }
    if (lane == 0) {
        p.n_accepted[b] = a + 1;
        if (p.counters != nullptr) {
            // passes, committed, proposed, accepted drafts, non-empty proposals, rows looked at (Section 6.5: OTE, SHR)
            atomicAdd(p.counters + 0, 1ull);
            atomicAdd(p.counters + 1, static_cast<unsigned long long>(a + 1));
            atomicAdd(p.counters + 2, static_cast<unsigned long long>(nd));
            atomicAdd(p.counters + 3, static_cast<unsigned long long>(a));
            atomicAdd(p.counters + 4, nd > 0 ? 1ull : 0ull);
            atomicAdd(p.counters + 5, static_cast<unsigned long long>((p.flags & kSkipUnusedRows) ? nd + 1 : K1));
        }
    }

    if (kMode != kTailVerifyOnly) {
        if (kMode == kTailResume || kWalkBeforeWait) {
            // the walk over the accepted draft prefix was done ahead of time
            if (a > 0) {
                const int src = a - 1;
                s = __shfl_sync(kFull, ps, src);
                L = __shfl_sync(kFull, pl, src);
                r.a.x = __shfl_sync(kFull, rj.a.x, src); r.a.y = __shfl_sync(kFull, rj.a.y, src);
                r.a.z = __shfl_sync(kFull, rj.a.z, src); r.a.w = __shfl_sync(kFull, rj.a.w, src);
                r.b.x = __shfl_sync(kFull, rj.b.x, src); r.b.y = __shfl_sync(kFull, rj.b.y, src);
                r.b.z = __shfl_sync(kFull, rj.b.z, src); r.b.w = __shfl_sync(kFull, rj.b.w, src);
            }
        } else {
            for (int t = 0; t < a; ++t) {
                const int c = __shfl_sync(kFull, d, t);
                walk_token(sam, c, s, L, r, lane);
            }
        }
        walk_token(sam, bonus, s, L, r, lane);
        int nn = 0;
        if (p.flags & kNoSpeculation) {
            if (lane < K) p.next_drafts[static_cast<long long>(b) * K + lane] = -1;
        } else {
            nn = emit_draft(sam, L, r, K, p.min_match, p.next_drafts + static_cast<long long>(b) * K, lane);
        }
        if (lane == 0) {
            p.state[b] = s;
            p.matched_len[b] = L;
            if (p.acc_epoch != nullptr) {
                // inside the argmax kernel: whoever still classifies rows of this stream must not take the next proposal's
                // length (next_n_draft may be n_draft itself) for this one's
                p.acc_epoch[b] = epoch;
                __threadfence();
            }
            p.next_n_draft[b] = nn;
        }
        if (p.next_list != nullptr) {
            // The rows the next step will need from this stream go into the next row list.  The argmax kernel that
            // read the current list has finished (this kernel waited for it), so the list is rewritten in place; order
            // does not matter.  One 64-bit atomic per stream both reserves the stream's places and counts the streams
            // that have come by; the last one publishes the total and leaves the word zero for the next step.  The
            // reader is the next kernel in the stream, so no ordering is needed between a stream's entries and the total.
            const int need = nn + 1;
            unsigned long long old = 0ull;
            unsigned long long* accum = reinterpret_cast<unsigned long long*>(p.list_meta + kListAccum);
            if (lane == 0) old = atomicAdd(accum, (1ull << 32) | static_cast<unsigned long long>(need));
            old = __shfl_sync(kFull, old, 0);
            const int base = static_cast<int>(old & 0xFFFFFFFFull);
            for (int j = lane; j < need; j += 32) p.next_list[base + j] = static_cast<int>(row0) + j;
            if (lane == 0 && static_cast<int>(old >> 32) == p.B - 1) {
                p.list_meta[kListCount] = base + need;
                p.list_meta[kListSig] = row_list_sig(p.B, K);
                *accum = 0ull;
            }
        }
    }
}

// kDependent: launched as a programmatic dependent of the argmax kernel (waits for that grid inside);
// otherwise an ordinary launch behind whatever produced the row results.
template <int kMode, bool kDependent = true>
__global__ void __launch_bounds__(128)
accept_kernel(DeviceSam sam, AcceptArgs p) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (b >= p.B) return;
    accept_stream<kMode, kDependent>(sam, p, b, lane);
}

__global__ void __launch_bounds__(32 * kMaxSlots)
multi_step_kernel(AcceptArgs p, MultiArgs q) {
    __shared__ float score[kMaxSlots];
    __shared__ int ok[kMaxSlots];
    __shared__ int winner, sh_a, sh_bonus;
    const int b = blockIdx.x;
    const int m = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int K = p.K;
    const long long at = static_cast<long long>(b) * q.M + m;
    // what does not depend on the argmax kernel
    const int member = q.slots[at];
    const bool live = member >= 0 && member < q.n_members;
    int s = 0, L = 0;
    RecRegs r = root_rec();
    DeviceSam sam;
    if (live) {
        sam = q.table[member];
        s = q.state[at];
        L = q.matched_len[at];
        sanitize_stream_state(sam, s, L);
        if (s != 0) r = load_rec(sam, s);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (m == 0) {
        int a = 0, bonus = 0;
        accept_stream<kTailVerifyOnly>(DeviceSam{}, p, b, lane, &a, &bonus);
        if (lane == 0) { sh_a = a; sh_bonus = bonus; }
    }
    __syncthreads();
    const int a = sh_a, bonus = sh_bonus;
    if (live) {
        if (a > 0) {                                   // resume after the accepted prefix
            s = __ldcg(q.pre_state + at * K + (a - 1));
            L = __ldcg(q.pre_len + at * K + (a - 1));
            r = (s > 0 && s < sam.n_states) ? load_rec(sam, s) : root_rec();
            if (!(s > 0 && s < sam.n_states)) { s = 0; L = 0; }
        }
        walk_token(sam, bonus, s, L, r, lane);
        if (lane == 0) {
            q.state[at] = s;
            q.matched_len[at] = L;
        }
    }
    if (lane == 0) {
        ok[m] = live && L >= p.min_match;
        score[m] = live ? q.weights[at] * static_cast<float>(L) : 0.0f;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int w = -1;
        float best = 0.0f;
        for (int x = 0; x < q.M; ++x)
            if (ok[x] && (w < 0 || score[x] > best)) { w = x; best = score[x]; }
        winner = w;
        q.chosen[b] = w;
        if (w < 0) p.next_n_draft[b] = 0;
    }
    __syncthreads();
    if (winner == m) {
        const int nd = emit_draft(sam, L, r, K, p.min_match, p.next_drafts + static_cast<long long>(b) * K, lane);
        if (lane == 0) p.next_n_draft[b] = nd;
    } else if (winner < 0 && m == 0 && lane < K) {
        p.next_drafts[static_cast<long long>(b) * K + lane] = -1;
    }
}

}  // namespace samb200
