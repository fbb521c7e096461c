// Internal (not part of the C ABI): host-side automaton, device layout description.
#pragma once
#include <cstdint>
#include <vector>

#include "sam.h"

namespace samb200 {

// One 32-byte record per state = one DRAM/L2 sector per state visit.
//   deg == 1 : e[0]=tok0 e[1]=dst0                      (transition stored inline)
//   deg == 2 : e[0]=tok0 e[1]=dst0 e[2]=tok1 e[3]=dst1  (both inline, ascending)
//   3 <= deg <= kSortedRowMax : e[0]=offset of the state's row in the wide-edge array (units of one
//              edge), e[1] = -1; the row holds the deg transitions ascending by token - one warp-wide
//              read finds any of them
//   deg > kSortedRowMax : e[0]=offset, e[1]=log2 of the row's capacity; the row is an open-addressing
//              hash table (linear probing from hash_slot(tok), empty slots have tok = -1, never more
//              than half full, nothing is ever deleted) - one warp-wide read of 32 consecutive slots
//              finds a transition or proves its absence in all but freak cases
//   root     : transitions come from the dense root table, e[] unused
struct StateRec {
    int32_t len, link, firstpos, deg;
    int32_t e[4];
};
static_assert(sizeof(StateRec) == 32, "one sector per state");

struct Edge { int32_t tok, dst; };

constexpr int32_t kSortedRowMax = 32;

#ifdef __CUDACC__
#define SAM_HD __host__ __device__ __forceinline__
#else
#define SAM_HD inline
#endif
// First slot probed for token tok in a hash row of 2^log2cap slots (multiplicative hashing).
SAM_HD uint32_t hash_slot(int32_t tok, int32_t log2cap) {
    return (static_cast<uint32_t>(tok) * 0x9E3779B1u) >> (32 - log2cap);
}
// Capacity (log2) of a fresh hash row for deg transitions: the smallest power of two >= room * deg
// (room = 2 for an index that never grows; 4 for one that does, so that a row can double its population
// before it has to move).
SAM_HD int32_t hash_log2cap(int32_t deg, int32_t room) {
    int32_t l = 7;
    while ((int64_t(1) << l) < int64_t(room) * deg) ++l;
    return l;
}

// Where things sit inside the caller's device blob (byte offsets, 256-byte aligned).
// A growing index sizes every section for its capacity and adds a staging area for updates.
struct DeviceLayout {
    int64_t rec_off = 0, edge_off = 0, root_off = 0, corpus_off = 0, stage_off = 0, total = 0;
    int64_t n_states = 0, n_wide_edges = 0, root_span = 0, n_corpus = 0, stage_bytes = 0;
    int64_t ring_off = 0, ctrl_off = 0;      // growing index: slots for updates copied ahead of time; a few control words
};

// Updates of a growing index that are small enough (the usual case between two decoding steps) travel as one flat
// buffer: [record ids][records][row descriptors][row edges][root tokens][root destinations][appended text].
struct StagedLayout {
    int64_t off_ids = 0, off_recs = 0, off_descs = 0, off_edges = 0, off_rtok = 0, off_rdst = 0, off_tail = 0, total = 0;
    int32_t n_rec = 0, n_seg = 0, n_root = 0, n_tail = 0;
};
constexpr int kRingSlots = 8;                          // updates that can wait on the device for sam_sync
constexpr int64_t kRingSlotBytes = int64_t(1) << 20;   // largest update that takes this route
constexpr int kDirectRowEdges = 2048;                  // rows at least this long are copied straight to their place

// Pointers handed to kernels by value.
struct DeviceSam {
    const StateRec* rec;
    const Edge* wide;
    const int32_t* root_dst;  // [root_span], -1 = no transition
    const int32_t* corpus;    // [n_corpus]
    int32_t root_span;
    int32_t n_states;
    int32_t n_sep;
    int32_t pad_;
    int64_t n_corpus;
    int32_t seps[SAM_MAX_SEPARATORS];
};

// ---- growing index (appending verified tokens; Section 5.4.2 / 5.4.3) --------------------------
// What changed on the host since the device image was last brought up to date.
struct WideSeg {
    int64_t dst_off;   // first edge of the row in the device's wide array
    int64_t src_off;   // first edge of the row in Delta::seg_edges
    int32_t len;
};
struct Delta {
    bool full = false;                       // whole image (first upload, or after the wide rows were compacted)
    int status = SAM_OK;
    std::vector<int32_t> rec_ids;            // states whose 32-byte record changed ...
    std::vector<StateRec> recs;              // ... and the new records
    std::vector<WideSeg> segs;               // wide rows to (re)write
    std::vector<Edge> seg_edges;
    std::vector<int32_t> root_tok, root_dst; // changed entries of the dense root table (one per token)
    int64_t corpus_off = 0;                  // appended text
    std::vector<int32_t> corpus_tail;
    int64_t n_states_after = 0, n_tokens_after = 0;
    // set by the builder thread when it has already sent the update to a ring slot of the device blob
    int staged_slot = -1;
    uint64_t staged_epoch = 0;
    StagedLayout staged;
    // full image only
    std::vector<StateRec> all_rec;
    std::vector<Edge> all_wide;
    std::vector<int32_t> all_root, all_corpus;
};
struct DynIndex;   // host-side state of a growing index (sam_dynamic.cpp)
struct UpdateRing; // CUDA objects of the asynchronous update path (sam_capi.cu)

}  // namespace samb200

struct sam_index {
    // flat automaton (host)
    std::vector<int32_t> len, link, firstpos;
    std::vector<int64_t> row_ptr;
    std::vector<int32_t> edge_tok, edge_dst;
    std::vector<int32_t> corpus;
    std::vector<int32_t> seps;
    samb200::DeviceLayout layout;
    // set by sam_upload
    void* device_buf = nullptr;
    samb200::DeviceSam dev{};
    // growing index only
    samb200::DynIndex* dyn = nullptr;
    int64_t updates_incremental = 0, updates_full = 0, update_bytes = 0;   // what sam_sync has applied so far
    // page-locked staging for small updates and the event that says when its last copy has left it (CUDA objects,
    // created by the first incremental update, released by sam_free)
    void* pinned_stage = nullptr;
    int64_t pinned_bytes = 0;
    void* stage_event = nullptr;
    // copy stream, page-locked slots and events with which the builder thread sends small updates ahead of sam_sync
    samb200::UpdateRing* ring = nullptr;
};

namespace samb200 {
// Online construction + CSR flattening. Returns SAM_OK / SAM_ERR_*.
int build_index(const int32_t* corpus, int64_t n, const int32_t* seps, int32_t n_sep, sam_index* out);
// Fills the packed host image of the device blob (rec / wide edges / root table); corpus is copied separately.
void pack_records(const sam_index& idx, StateRec* rec, Edge* wide, int32_t* root_dst);

// Growing index.  All of these are host-side; none touches the device.
int dyn_create(sam_index* idx, const int32_t* corpus, int64_t n, int64_t max_tokens, int32_t max_token_id);
void dyn_destroy(sam_index* idx);
int dyn_enqueue(sam_index* idx, const int32_t* tokens, int64_t n);     // hands tokens to the builder thread
int dyn_wait(sam_index* idx);                                          // until the builder thread has nothing left
bool dyn_pop_ready(sam_index* idx, Delta* out);                        // next finished update, in order
int dyn_full_image(sam_index* idx, Delta* out);                        // waits, drops queued updates, packs everything
int dyn_sizes(sam_index* idx, int64_t* n_states, int64_t* n_edges);    // waits; states / transitions right now
int dyn_refresh_csr(sam_index* idx);                                   // waits, refills the flat arrays for sam_export
void dyn_counts(sam_index* idx, int64_t* queued, int64_t* built);      // tokens handed in / tokens indexed on the host
int dyn_set_relayout_every(sam_index* idx, int64_t every);
// Layout of a small update's flat buffer, and the buffer itself (h holds layout.total bytes).
void staged_layout(const Delta& D, StagedLayout* out);
void staged_fill(const Delta& D, const StagedLayout& L, char* h);
// Called by the builder thread for every finished update: copies it towards the device if it can (sam_capi.cu).
void ring_stage_async(sam_index* idx, Delta* D);             // every k-th update becomes a whole image (0: never forced)
}  // namespace samb200
