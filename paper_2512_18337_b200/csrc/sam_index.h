// Internal (not part of the C ABI): host-side automaton, device layout description.
#pragma once
#include <cstdint>
#include <vector>

#include "sam.h"

namespace samb200 {

// One 32-byte record per state = one DRAM/L2 sector per state visit.
//   deg == 1 : e[0]=tok0 e[1]=dst0                      (transition stored inline)
//   deg == 2 : e[0]=tok0 e[1]=dst0 e[2]=tok1 e[3]=dst1  (both inline, ascending)
//   deg >= 3 : e[0]=offset of the state's row in the wide-edge array (units of one edge)
//   root     : transitions come from the dense root table, e[] unused
struct StateRec {
    int32_t len, link, firstpos, deg;
    int32_t e[4];
};
static_assert(sizeof(StateRec) == 32, "one sector per state");

struct Edge { int32_t tok, dst; };  // wide rows: ascending by tok

// Where things sit inside the caller's device blob (byte offsets, 256-byte aligned).
struct DeviceLayout {
    int64_t rec_off = 0, edge_off = 0, root_off = 0, corpus_off = 0, total = 0;
    int64_t n_states = 0, n_wide_edges = 0, root_span = 0, n_corpus = 0;
};

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
};

namespace samb200 {
// Online construction + CSR flattening. Returns SAM_OK / SAM_ERR_*.
int build_index(const int32_t* corpus, int64_t n, const int32_t* seps, int32_t n_sep, sam_index* out);
// Fills the packed host image of the device blob (rec / wide edges / root table); corpus is copied separately.
void pack_records(const sam_index& idx, StateRec* rec, Edge* wide, int32_t* root_dst);
}  // namespace samb200
