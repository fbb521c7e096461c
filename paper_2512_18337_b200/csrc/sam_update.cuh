// Device side of the growing index (sm_100a). Included only by sam_capi.cu.
//
// Updates arrive in the staging area of the device blob as flat lists and are scattered into the
// record array, the wide-edge array and the dense root table by the kernels below.  They run on the
// caller's stream between decoding steps, so no walk ever sees a half-applied update.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "sam_index.h"

namespace samb200 {

// rec[ids[i]] = recs[i]; one thread per record, two 16-byte stores.
__global__ void __launch_bounds__(256)
scatter_records_kernel(StateRec* __restrict__ rec, const int32_t* __restrict__ ids,
                       const StateRec* __restrict__ recs, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int4* src = reinterpret_cast<const int4*>(recs + i);
    int4* dst = reinterpret_cast<int4*>(rec + ids[i]);
    const int4 a = src[0], b = src[1];
    dst[0] = a;
    dst[1] = b;
}

struct SegDesc {
    long long dst_off;   // first edge of the row in the wide array
    int src_off;         // first edge of the row in the staged edge list
    int len;
};

// One warp per rewritten wide row.
__global__ void __launch_bounds__(256)
copy_rows_kernel(Edge* __restrict__ wide, const SegDesc* __restrict__ segs, const Edge* __restrict__ staged, int n) {
    const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n) return;
    const SegDesc g = segs[w];
    const int2* src = reinterpret_cast<const int2*>(staged + g.src_off);
    int2* dst = reinterpret_cast<int2*>(wide + g.dst_off);
    for (int k = lane; k < g.len; k += 32) dst[k] = src[k];
}

// root_dst[tok[i]] = dst[i]
__global__ void __launch_bounds__(256)
scatter_root_kernel(int32_t* __restrict__ root_dst, const int32_t* __restrict__ tok, const int32_t* __restrict__ dst,
                    int n, int span) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int t = tok[i];
    if (t >= 0 && t < span) root_dst[t] = dst[i];
}

// A whole small update in one launch: the staged buffer holds record ids and records, row descriptors and
// their edges, root entries and the appended text; every destination is written by exactly one thread (records,
// root entries, text) or one warp (rows), and the four parts touch different arrays.
struct UpdateArgs {
    StateRec* rec;
    Edge* wide;
    int32_t* root;
    int32_t* corpus;        // where the appended text goes
    const char* stage;
    long long off_ids, off_recs, off_descs, off_edges, off_rtok, off_rdst, off_tail;
    int n_rec, n_seg, n_root, n_tail, root_span;
};

// Optional tail of the update kernel: once every block has finished scattering, the block that finishes last moves
// the caller's stream states to the states that now hold their strings (what renormalize_kernel does), so that one
// launch is all that stands between an update and the next decoding step.  B == 0: no tail.
struct RenormTail {
    DeviceSam sam;            // the view AFTER the update (state count included)
    int B;
    int* state;               // [B] in place
    const int* matched_len;   // [B]
    unsigned* blocks_done;    // zero between launches
};

// Climb suffix links until len(link(s)) < L <= len(s).  `fresh` = read past L1 and the read-only path: the records
// may have been written moments ago by other blocks of the same kernel.
template <bool fresh>
__device__ __forceinline__ int renormalized_state(const DeviceSam& sam, int s, int L) {
    if (s <= 0 || s >= sam.n_states || L < 0) return s;      // the walk kernels reset such pairs themselves
    for (int hop = 0; hop < (1 << 30) && s != 0; ++hop) {
        const int link = fresh ? __ldcg(&sam.rec[s].link) : __ldg(&sam.rec[s].link);
        if (link < 0 || link >= sam.n_states) break;
        const int link_len = (link == 0) ? 0 : (fresh ? __ldcg(&sam.rec[link].len) : __ldg(&sam.rec[link].len));
        if (L > link_len) break;
        s = link;
    }
    return s;
}

__global__ void __launch_bounds__(256)
apply_update_kernel(UpdateArgs a, RenormTail t) {
    const int nthreads = gridDim.x * blockDim.x;
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    const int32_t* ids = reinterpret_cast<const int32_t*>(a.stage + a.off_ids);
    const StateRec* recs = reinterpret_cast<const StateRec*>(a.stage + a.off_recs);
    for (int i = gtid; i < a.n_rec; i += nthreads) {
        const int4* src = reinterpret_cast<const int4*>(recs + i);
        int4* dst = reinterpret_cast<int4*>(a.rec + ids[i]);
        const int4 x = src[0], y = src[1];
        dst[0] = x;
        dst[1] = y;
    }
    const SegDesc* segs = reinterpret_cast<const SegDesc*>(a.stage + a.off_descs);
    const Edge* staged = reinterpret_cast<const Edge*>(a.stage + a.off_edges);
    for (int w = gtid >> 5; w < a.n_seg; w += nthreads >> 5) {
        const SegDesc g = segs[w];
        const int2* src = reinterpret_cast<const int2*>(staged + g.src_off);
        int2* dst = reinterpret_cast<int2*>(a.wide + g.dst_off);
        for (int k = lane; k < g.len; k += 32) dst[k] = src[k];
    }
    const int32_t* rtok = reinterpret_cast<const int32_t*>(a.stage + a.off_rtok);
    const int32_t* rdst = reinterpret_cast<const int32_t*>(a.stage + a.off_rdst);
    for (int i = gtid; i < a.n_root; i += nthreads) {
        const int tk = rtok[i];
        if (tk >= 0 && tk < a.root_span) a.root[tk] = rdst[i];
    }
    const int32_t* tail = reinterpret_cast<const int32_t*>(a.stage + a.off_tail);
    for (int i = gtid; i < a.n_tail; i += nthreads) a.corpus[i] = tail[i];

    if (t.B > 0) {
        __shared__ int is_last;
        __threadfence();                      // this thread's writes before the block's arrival
        __syncthreads();
        if (threadIdx.x == 0) is_last = (atomicAdd(t.blocks_done, 1u) == gridDim.x - 1);
        __syncthreads();
        if (is_last) {
            __threadfence();                  // every block has arrived: its writes are visible from here on
            for (int b = threadIdx.x; b < t.B; b += blockDim.x) {
                const int s0 = t.state[b];
                const int s = renormalized_state<true>(t.sam, s0, t.matched_len[b]);
                if (s != s0) t.state[b] = s;
            }
            if (threadIdx.x == 0) *t.blocks_done = 0u;
        }
    }
}

// After the text has grown, a stream's string of length L may belong to a state that was split off
// its old one: the state of a string is the one with len(link(s)) < L <= len(s) (renormalized_state).
// One thread per stream.
__global__ void __launch_bounds__(128)
renormalize_kernel(DeviceSam sam, int B, int* __restrict__ state, const int* __restrict__ matched_len) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int s0 = state[b];
    const int s = renormalized_state<false>(sam, s0, matched_len[b]);
    if (s != s0) state[b] = s;
}

// The same for composite drafting: only the slots that name `member` are touched (slots, state and
// matched_len are [n] = B * M entries).
__global__ void __launch_bounds__(128)
renormalize_slots_kernel(DeviceSam sam, int member, int n, const int* __restrict__ slots, int* __restrict__ state,
                         const int* __restrict__ matched_len) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n || slots[i] != member) return;
    const int s0 = state[i];
    const int s = renormalized_state<false>(sam, s0, matched_len[i]);
    if (s != s0) state[i] = s;
}

}  // namespace samb200
