// Vocabulary argmax, bulk-copy pipelined variant (sm_100a). Included only by sam_capi.cu.
//
// One persistent CTA per SM.  A producer thread streams row tiles from HBM into a ring of
// shared-memory stages with 1-D bulk asynchronous copies (cp.async.bulk, completion counted on
// an mbarrier); the consumer warps reduce the tiles straight out of shared memory.  Loads cost
// no issue slots and no registers, ~190 KB per SM are in flight, and the reduction of one tile
// overlaps the copies of the following ones.  Requires 16-byte aligned rows (base and stride) of at
// least one 16-byte vector; the direct-load kernel covers everything else.
//
// How the consumer warps share the tiles depends on the tile size (BulkPlan, chosen by the host).  A tile
// costs the consumers 0.58 us whatever its size - waking up on the barrier, the vote, locating the new
// maximum, releasing the stage - beside 0.69 us per 64 KB (measured with eight warps on every tile).  With
// tiles of about 60 KB (a 304 KB row cut in five) that keeps pace with HBM, and eight warps work on one tile
// after the other.  With smaller tiles (the 76 KB row pieces of a vocabulary shard cut in two) it does not:
// there the twelve consumer warps form three groups, tile k goes to group k mod 3, and the fixed cost of one
// group's tile runs while the other groups are busy with theirs; the ring then has as many stages as fit
// (five of 38 KB), so that the bytes in flight stay the same.
//
// The consumer warps never touch global memory for their results: when a row (or the CTA's part of
// it) is finished, each warp leaves its candidate in a small ring in shared memory and moves on.
// A finisher warp combines the eight candidates of up to 32 rows at a time (one row per lane) and
// publishes them with one 64-bit atomic max per row, so that the round trips to L2 stay off the
// streaming path.
//
// Fused tail.  When the host asks for it, the accept step of a stream (decode the row results,
// longest matching prefix, follow the model's own token, next draft) runs inside this kernel as
// soon as the rows it needs are complete.  It needs rows 0 .. n_draft[b] only (the rows behind the proposal
// are reported, nothing depends on them), so every CTA takes the used rows of its share first and the
// others afterwards: the accept steps then run under the second half of the stream instead of after it.
// A finished row is complete at once when the CTA had all its tiles; a row shared with the neighbouring
// CTA is complete when a counter says so.  A complete used row adds one to its stream's counter, the
// addition that completes the stream puts it into a queue in the CTA's shared memory, and idle warps of
// that CTA (the walk-ahead warps, the finisher and the consumer warps once their work is done) take
// streams from the queue; a complete row behind the proposal is decoded into argmax_out by the finisher
// itself.  Nobody waits for another CTA, so the scheme needs no co-residency.
//
// Every wait on an mbarrier is bounded: after kMaxPolls unsuccessful polls the waiting thread
// raises the CTA's abort flag and the status word in global memory, all roles leave their
// loops, the producer waits (bounded again) for copies still in flight, and the CTA exits.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <type_traits>

#include "sam_kernels.cuh"

namespace samb200 {

#ifndef SAM_BULK_TILE_VEC
#define SAM_BULK_TILE_VEC 4096
#endif
#ifndef SAM_BULK_STAGES
#define SAM_BULK_STAGES 3
#endif
constexpr int kBulkTileVec = SAM_BULK_TILE_VEC;        // largest tile in 16-byte vectors (64 KB)
constexpr int kBulkTileBytes = kBulkTileVec * 16;
constexpr int kBulkStages = SAM_BULK_STAGES;           // the ring holds kBulkStages * kBulkTileBytes (<= ~200 KB) ...
constexpr int kBulkRingBytes = kBulkStages * kBulkTileBytes;
constexpr int kMaxStages = 8;                          // ... cut into up to kMaxStages stages when the tiles are small
#ifndef SAM_BULK_CONSUMER_WARPS
#define SAM_BULK_CONSUMER_WARPS 12
#endif
constexpr int kBulkConsumerWarps = SAM_BULK_CONSUMER_WARPS;
constexpr int kBulkConsumers = kBulkConsumerWarps * 32;
constexpr int kWideGroupWarps = 8;                     // one group of eight warps on every tile (large tiles)
constexpr int kSmallGroupWarps = 4;                    // groups of four warps taking tiles in turn (small tiles):
constexpr int kSmallGroups = kBulkConsumerWarps / kSmallGroupWarps;   // three of them
#ifndef SAM_BULK_SMALL_TILE_BYTES
#define SAM_BULK_SMALL_TILE_BYTES (48 * 1024)
#endif
constexpr int kSmallTileBytes = SAM_BULK_SMALL_TILE_BYTES;   // below this a tile counts as small
static_assert(kWideGroupWarps <= kBulkConsumerWarps && kSmallGroups * kSmallGroupWarps <= kBulkConsumerWarps, "consumer warps");

// How the rows are tiled and how the consumer warps share the tiles (filled in by bulk_plan on the host).
struct BulkPlan {
    int tiles_per_row;     // a row is cut into this many tiles of tile_vec vectors (the last one may be shorter)
    int tile_vec;
    int n_stages;          // stages of stage_bytes bytes in the ring
    int stage_bytes;
    int n_groups;          // consumer groups; tile k of a CTA is reduced by group k mod n_groups
    int group_warps;       // warps per group
};
inline BulkPlan bulk_plan(int V) {
    BulkPlan p;
    const long long nvec = V / 8;
    p.tiles_per_row = static_cast<int>((nvec + kBulkTileVec - 1) / kBulkTileVec);
    p.tile_vec = static_cast<int>((nvec + p.tiles_per_row - 1) / p.tiles_per_row);   // nearly equal tiles
    p.stage_bytes = (p.tile_vec * 16 + 127) & ~127;
    const bool small = p.stage_bytes < kSmallTileBytes;
    p.n_groups = small ? kSmallGroups : 1;
    p.group_warps = small ? kSmallGroupWarps : kWideGroupWarps;
    p.n_stages = kBulkRingBytes / p.stage_bytes;
    if (p.n_stages > kMaxStages) p.n_stages = kMaxStages;
    return p;
}
constexpr int kBulkWalkerWarps = 2;                    // spare warps that walk ahead along the drafts
constexpr int kBulkThreads = kBulkConsumers + 64 + kBulkWalkerWarps * 32;   // consumers, producer, finisher, walkers
constexpr int kRowSlots = 64;                          // ring of per-row candidate slots (consumers -> finisher)
constexpr uint32_t kMaxPolls = 1u << 22;
constexpr int kQueueCap = 1024;                        // streams one CTA can be handed (host checks the bound)
constexpr size_t kBulkCtrlOff = static_cast<size_t>(kBulkRingBytes);
constexpr size_t kBulkQueueOff = kBulkCtrlOff + 1024;
constexpr size_t kBulkCandOff = kBulkQueueOff + kQueueCap * 4;
constexpr int kOrderCap = 1024;                        // rows of a CTA that can be taken in another order than they lie
constexpr size_t kBulkOrderOff = kBulkCandOff + static_cast<size_t>(kRowSlots) * kBulkConsumerWarps * 8;
constexpr size_t kBulkSmemBytes = kBulkOrderOff + static_cast<size_t>(kOrderCap) * 4;


__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Global -> shared bulk copy of `bytes` (multiple of 16, both addresses 16-byte aligned) into this
// CTA's own shared memory; completion is signalled on `bar` as transferred bytes.
// The logits are read exactly once, so their lines are marked evict-first in L2 (`policy`): the
// automaton records, the root table and the corpus lines that the walks touch stay resident.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar,
                                          uint64_t policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// Poll with a limit; also gives up early when another thread of the CTA has raised `abort`.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort) {
    for (uint32_t i = 0; i < kMaxPolls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i >= 4096u) __nanosleep(64);
        if ((i & 1023u) == 1023u && *abort) return false;
    }
    return false;
}

struct BulkShared {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    long long issued;                 // tiles the producer has issued copies for
    int abort;
    int q_tail;                       // streams pushed into the queue
    int q_head;                       // tickets handed to worker warps
    int fin_rows;                     // rows of this CTA the finisher has published
    int fin_finished;                 // the finisher has left its loop: no pushes after that
    int prog[kBulkConsumerWarps];     // rows each consumer warp has handed over
    int n_used;                       // accept step inside the kernel: the first n_used rows the CTA takes are used rows
    int u_of[32];                     // ... and the number of used rows of every stream of the CTA's share
};
static_assert(sizeof(BulkShared) <= 1024, "control block");

// Fused accept step (see the file header).  `done[b]` counts the contributions to stream b that have arrived and
// `rowcnt[r]` the tiles of a shared row; both are zero between calls.
struct FusedTail {
    AcceptArgs args;
    int* done;       // [B] contributions that have arrived: the stream's used rows (0..n_draft), + 1 for its walk-ahead
    int* rowcnt;     // [R] tiles reduced so far of a row that two CTAs share
    int prewalk;     // 1: the walk-ahead of a stream counts as one of its contributions
    int mode;        // 0 = off, else kTailVerifyOnly + 1 or kTailResume + 1
    int* launch_words;   // [0] launches through this scratch so far, [1] CTAs of the current launch that have left
};
// Rows 0 .. n_draft[b] of stream b are the ones its accept step needs ("used"); returns their number.  n_draft is read
// past the read-only path: the accept step of the stream may overwrite it in this very launch (next_n_draft may be the
// same array).
__device__ __forceinline__ int used_rows_of(const AcceptArgs& a, int b) {
    return ((a.flags & kNoSpeculation) ? 0 : max(0, min(__ldcg(a.n_draft + b), a.K))) + 1;
}
// The same for a row that completes at an unknown time: once the stream's accept step has run in this launch, n_draft[b]
// may already hold the NEXT proposal's length, and whatever completes after that step is a row behind the proposal
// (the step waited for all the others).  The step writes the launch's number into acc_epoch[b], then a fence, then
// n_draft; here the order is n_draft, fence, acc_epoch - so a count taken from n_draft is the old one whenever the
// launch's number is not seen yet.
__device__ __forceinline__ int used_rows_now(const FusedTail& ft, int epoch, int b) {
    const int u = used_rows_of(ft.args, b);
    __threadfence();
    return (__ldcg(ft.args.acc_epoch + b) == epoch) ? 0 : u;
}

__device__ __forceinline__ int ld_volatile_s32(const int* p) { return *reinterpret_cast<const volatile int*>(p); }
__device__ __forceinline__ void st_volatile_s32(int* p, int v) { *reinterpret_cast<volatile int*>(p) = v; }

__device__ __forceinline__ void fused_accept(const DeviceSam& sam, const FusedTail& ft, int epoch, int b, int lane) {
    __threadfence();                 // order the reads below after the counter observation
    if (ft.mode == kTailResume + 1) accept_stream<kTailResume>(sam, ft.args, b, lane, nullptr, nullptr, epoch);
    else accept_stream<kTailVerifyOnly>(sam, ft.args, b, lane, nullptr, nullptr, epoch);
    if (lane == 0) ft.done[b] = 0;
}

// Idle warps serve the CTA's queue until the finisher has left its loop and the queue is drained.
// Each round takes one ticket; a ticket beyond the final tail means there is no more work.
__device__ __forceinline__ void serve_queue(const DeviceSam& sam, const FusedTail& ft, int epoch, BulkShared* sh,
                                            const int* queue, volatile int* abort, int* status, int lane) {
    for (;;) {
        int b = -1;
        if (lane == 0) {
            const int ticket = atomicAdd(&sh->q_head, 1);
            uint32_t polls = 0;
            for (;;) {
                if (ticket < kQueueCap) {
                    b = ld_volatile_s32(queue + ticket);
                    if (b >= 0) break;
                }
                const bool finished = ld_volatile_s32(&sh->fin_finished) != 0;
                if (finished && ticket >= ld_volatile_s32(&sh->q_tail)) { b = -1; break; }
                if (*abort) { b = -1; break; }
                if (++polls > kMaxPolls) {
                    *abort = 1;
                    atomicExch(status, kStatusWaitTimeout);
                    b = -1;
                    break;
                }
                __nanosleep(128);
            }
        }
        b = __shfl_sync(kFull, b, 0);
        if (b < 0) return;
        fused_accept(sam, ft, epoch, b, lane);
    }
}

__global__ void __launch_bounds__(kBulkThreads, 1)
argmax_bulk_kernel(const __nv_bfloat16* __restrict__ logits, long long stride, long long R, int V,
                   const __grid_constant__ BulkPlan plan, unsigned long long* __restrict__ keys,
                   int* __restrict__ status, const __grid_constant__ DeviceSam sam,
                   const __grid_constant__ PreWalk pw, const __grid_constant__ FusedTail ft,
                   const __grid_constant__ RowMap rm) {
    const int tiles_per_row = plan.tiles_per_row, tile_vec = plan.tile_vec, ns = plan.n_stages;
    const int n_cons = plan.n_groups * plan.group_warps;                      // consumer warps that take part
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* stage_base = smem_raw;                                      // ns stages of plan.stage_bytes
    BulkShared* sh = reinterpret_cast<BulkShared*>(smem_raw + kBulkCtrlOff);
    int* queue = reinterpret_cast<int*>(smem_raw + kBulkQueueOff);
    unsigned long long* cand = reinterpret_cast<unsigned long long*>(smem_raw + kBulkCandOff);   // [kRowSlots][warps]
    int* order = reinterpret_cast<int*>(smem_raw + kBulkOrderOff);             // [kOrderCap] the CTA's rows in the order it takes them

    // the accept kernel may be scheduled now; it waits for this grid before it reads any result
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // with a row list the number of rows is only known on the device, and a CTA's share may be empty
    const long long n_all = (rm.list != nullptr) ? listed_rows(rm, R) : R;
    const long long total = n_all * tiles_per_row;
    const long long t0 = total * blockIdx.x / gridDim.x;
    const long long t1 = total * (blockIdx.x + 1) / gridDim.x;
    const long long row_first = t0 / tiles_per_row;      // position in the list (or the row itself without one)
    const int n_rows = (t1 > t0) ? static_cast<int>((t1 - 1) / tiles_per_row - row_first + 1) : 0;   // rows this CTA touches
    const int nvec_row = V >> 3;               // whole 16-byte vectors per row (rows are 16-byte aligned)
    const int ragged = V & 7;                  // trailing elements read with plain loads

    if (threadIdx.x == 0) {
        for (int s = 0; s < ns; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->empty[s], plan.group_warps);
        }
        sh->abort = 0;
        sh->issued = 0;
        sh->q_tail = 0;
        sh->q_head = 0;
        sh->fin_rows = 0;
        sh->fin_finished = 0;
        for (int w = 0; w < kBulkConsumerWarps; ++w) sh->prog[w] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (ft.mode != 0)
        for (int i = threadIdx.x; i < kQueueCap; i += blockDim.x) queue[i] = -1;
    // With the accept step inside the kernel: the used rows (0 .. n_draft) of the CTA's share first, the rows behind the
    // proposals afterwards.  One lane per stream of the share counts the stream's used and other rows inside the share,
    // a warp-wide running sum gives every stream its two places, and the lane writes its stream's rows there.
    // the number of this launch: one more than the launches that have gone through the scratch (a replayed graph counts too)
    const int epoch = (ft.mode != 0) ? __ldcg(ft.launch_words) + 1 : 0;
    const int K1 = ft.args.K + 1;
    const long long b_first = (ft.mode != 0) ? row_first / K1 : 0;
    const int n_streams = (ft.mode != 0 && n_rows > 0) ? static_cast<int>((row_first + n_rows - 1) / K1 - b_first + 1) : 0;
    const bool ordered = ft.mode != 0 && plan.n_groups == 1 && n_rows > 0 && n_rows <= kOrderCap && n_streams <= 32;
    if (ordered && warp == 0) {
        int used = 0, rest = 0, j_lo = 0, j_hi = 0, u = 0;
        if (lane < n_streams) {
            const long long b = b_first + lane;
            j_lo = static_cast<int>(max(0ll, row_first - b * K1));
            j_hi = static_cast<int>(min(static_cast<long long>(K1), row_first + n_rows - b * K1));      // exclusive
            u = used_rows_now(ft, epoch, static_cast<int>(b));
            used = max(0, min(u, j_hi) - j_lo);
            rest = (j_hi - j_lo) - used;
        }
        int used_before = used, rest_before = rest;                // inclusive running sums over the lanes
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int a = __shfl_up_sync(kFull, used_before, d), c = __shfl_up_sync(kFull, rest_before, d);
            if (lane >= d) { used_before += a; rest_before += c; }
        }
        const int all_used = __shfl_sync(kFull, used_before, 31);
        used_before -= used;
        rest_before -= rest;
        if (lane == 0) sh->n_used = all_used;
        if (lane < n_streams) {
            sh->u_of[lane] = u;
            const int base = static_cast<int>((b_first + lane) * K1 - row_first);     // the stream's row 0 as a row of the share
            for (int j = j_lo; j < j_hi; ++j) {
                const int at = (j < u) ? used_before + (j - j_lo) : all_used + rest_before + (j - max(j_lo, u));
                order[at] = base + j;
            }
        }
    }
    if (ft.mode != 0 && !ordered && n_rows > 0 && threadIdx.x == 0)
        atomicExch(status, kStatusQueueOverflow);      // the host enables the accept step only for shares that can be ordered
    __syncthreads();
    volatile int* abort = &sh->abort;
    // The i-th row this CTA takes (as a position: in the list, or the row itself), and which of its tiles are the CTA's.
    auto seq_row = [&](int i) -> long long { return row_first + (ordered ? order[i] : i); };
    auto tiles_of = [&](long long r, int& lo, int& hi) {
        const long long first = r * tiles_per_row;
        lo = (t0 > first) ? static_cast<int>(t0 - first) : 0;
        hi = (t1 - first < tiles_per_row) ? static_cast<int>(t1 - first) : tiles_per_row;
    };
    // a row named by a list is clamped into the logits: a stale or foreign list can give wrong results, never a fault
    auto actual_row = [&](long long pos) -> long long {
        if (rm.list == nullptr) return pos;
        const long long r = __ldg(rm.list + pos);
        return r < 0 ? 0 : (r >= R ? R - 1 : r);
    };

    if (warp == kBulkConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            long long it = 0;
            bool ok = true;
            int s = 0;
            uint32_t use = 0;
            const uint64_t policy = l2_evict_first_policy();
            for (int i = 0; i < n_rows && ok; ++i) {
                const long long row = seq_row(i);
                int tile, tile_hi;
                tiles_of(row, tile, tile_hi);
                // with a row list the row number is fetched before the wait, off the path of the copy
                const __nv_bfloat16* src = logits + actual_row(row) * stride;
                for (; tile < tile_hi; ++tile, ++it) {
                    if (!mbar_wait_bounded(&sh->empty[s], (use & 1u) ^ 1u, abort)) { ok = false; break; }
                    const int v0 = tile * tile_vec;
                    const int nv = max(0, min(tile_vec, nvec_row - v0));
                    const uint32_t bytes = static_cast<uint32_t>(nv) * 16u;
                    mbar_arrive_expect_tx(&sh->full[s], bytes);
                    bulk_load(stage_base + static_cast<size_t>(s) * plan.stage_bytes,
                              reinterpret_cast<const uint4*>(src) + v0, bytes, &sh->full[s], policy);
                    if (++s == ns) { s = 0; ++use; }
                }
            }
            sh->issued = it;
            if (!ok) {
                *abort = 1;
                atomicExch(status, kStatusWaitTimeout);
            }
        }
    } else if (warp == kBulkConsumerWarps + 1) {
        // ------------------------------------------------------------------ finisher
        int done_rows = 0;
        uint32_t polls = 0;
        while (done_rows < n_rows) {
            int p = (lane < n_cons) ? ld_volatile_s32(&sh->prog[lane]) : 0x7fffffff;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) p = min(p, __shfl_xor_sync(kFull, p, d));
            if (p <= done_rows) {                      // nothing new: every warp must have handed the row over
                if (__shfl_sync(kFull, (lane == 0) ? *abort : 0, 0)) break;     // one reading for the whole warp
                if (++polls > kMaxPolls) {
                    if (lane == 0) {
                        *abort = 1;
                        atomicExch(status, kStatusWaitTimeout);
                    }
                    break;
                }
                __nanosleep(64);
                continue;
            }
            polls = 0;
            __threadfence_block();                     // candidates were written before the progress counters
            const int n = min(32, p - done_rows);
            if (lane < n) {
                const int i = done_rows + lane;
                const long long pos = (plan.n_groups == 1) ? seq_row(i) : row_first + i;
                const long long row = actual_row(pos);
                const unsigned long long* c = cand + static_cast<size_t>(i % kRowSlots) * kBulkConsumerWarps;
                unsigned long long k = 0ull;
#pragma unroll
                for (int w = 0; w < kBulkConsumerWarps; ++w) {
                    const unsigned long long x = (w < n_cons) ? c[w] : 0ull;
                    k = (x > k) ? x : k;
                }
                if (ft.mode == 0) {
                    if (k != 0ull) atomicMax(keys + row, k);
                } else {
                    int lo, hi;
                    tiles_of(pos, lo, hi);
                    const int seg = hi - lo;           // tiles of the row this CTA reduced
                    bool complete = seg == tiles_per_row;      // the row is this CTA's alone: k is its result
                    if (!complete) {
                        // shared with the neighbouring CTA: results meet in the row's word, a counter tells who came last
                        if (k != 0ull) atomicMax(keys + row, k);
                        __threadfence();
                        complete = atomicAdd(ft.rowcnt + row, seg) + seg == tiles_per_row;
                        if (complete) {
                            __threadfence();
                            k = __ldcg(keys + row);
                            ft.rowcnt[row] = 0;
                        }
                    }
                    if (complete) {
                        // used or not was settled when the CTA laid out its order (and cannot change for a row that was
                        // still missing then): no look at n_draft here, which the stream's accept step may have rewritten
                        const int b = static_cast<int>(row / K1);
                        if (i < sh->n_used) {
                            const int u = sh->u_of[b - static_cast<int>(b_first)];
                            // a row the stream's accept step needs: its word stays for that step, the stream counts it
                            if (seg == tiles_per_row) keys[row] = k;
                            __threadfence();               // the word first, then the count
                            if (atomicAdd(ft.done + b, 1) + 1 == u + ft.prewalk) {
                                __threadfence();
                                const int slot = atomicAdd(&sh->q_tail, 1);
                                if (slot < kQueueCap) st_volatile_s32(queue + slot, b);
                                else atomicExch(status, kStatusQueueOverflow);   // the host sizes the grid so that this cannot happen
                            }
                        } else {
                            // a row behind the proposal: nothing waits for it, it is reported from here
                            ft.args.argmax_out[row] = (k != 0ull) ? static_cast<int>(0xFFFFFFFFu - static_cast<unsigned>(k)) : 0;
                            if (seg != tiles_per_row) keys[row] = 0ull;
                        }
                    }
                }
            }
            __syncwarp();
            done_rows += n;
            if (lane == 0) {
                __threadfence_block();                 // slots are free again only after they have been read
                st_volatile_s32(&sh->fin_rows, done_rows);
            }
        }
        if (ft.mode != 0) {
            if (lane == 0) {
                __threadfence_block();                 // pushes before the "no more pushes" flag
                st_volatile_s32(&sh->fin_finished, 1);
            }
            __syncwarp();
            serve_queue(sam, ft, epoch, sh, queue, abort, status, lane);
        }
    } else if (warp > kBulkConsumerWarps + 1) {
        // ------------------------------------------------------------------ walk-ahead warps
        if (pw.enabled) {
            const int w = warp - kBulkConsumerWarps - 2;
            const int per_stream = pw.M > 0 ? pw.M : 1;
            for (int at = blockIdx.x * kBulkWalkerWarps + w; at < pw.B * per_stream; at += gridDim.x * kBulkWalkerWarps) {
                const int b = at / per_stream;
                if (pw.M > 0) {
                    // composite drafting: this slot's own automaton (an empty slot has nothing to walk)
                    const int member = __ldg(pw.slots + at);
                    if (member >= 0 && member < pw.n_members) {
                        const DeviceSam own = pw.table[member];
                        prewalk_stream(own, pw, b, at, lane);
                    }
                    continue;
                }
                prewalk_stream(sam, pw, b, at, lane);
                if (ft.mode != 0) {
                    // the walk-ahead is one of the stream's contributions; if it happens to be the last, finish here
                    int last = 0;
                    if (lane == 0) {
                        __threadfence();
                        last = (atomicAdd(ft.done + b, 1) + 1 == used_rows_of(ft.args, b) + ft.prewalk);
                    }
                    __syncwarp();
                    if (__shfl_sync(kFull, last, 0)) fused_accept(sam, ft, epoch, b, lane);
                }
            }
        }
        if (ft.mode != 0) serve_queue(sam, ft, epoch, sh, queue, abort, status, lane);
    } else {
        // ------------------------------------------------------------------ consumers
        bool ok = true;
        float best = __int_as_float(0xff800000);          // -inf: only strictly greater values are candidates
        int best_idx = -1;
        bool first_nan = false;                           // element 0 of the current row is NaN (seen by one thread only)
        // Hands this warp's candidate for the CTA's row number i over to the finisher: into the row's slot, then the
        // progress counter.  Every taking-part consumer warp hands over every row of the CTA, in order.
        auto hand_over = [&](int i) -> bool {
            unsigned long long k = (best_idx >= 0) ? pack_candidate(best, static_cast<unsigned>(best_idx + rm.v_offset)) : 0ull;
            if (first_nan) k = kCandidateFirstIsNaN;
            k = warp_max_u64(k);
            int good = 1;
            if (lane == 0) {
                uint32_t polls = 0;
                while (i - ld_volatile_s32(&sh->fin_rows) >= kRowSlots) {     // ring full: the finisher is behind
                    if (*abort || ++polls > kMaxPolls) { good = 0; break; }
                    __nanosleep(64);
                }
                if (good) {
                    cand[static_cast<size_t>(i % kRowSlots) * kBulkConsumerWarps + warp] = k;
                    __threadfence_block();
                    st_volatile_s32(&sh->prog[warp], i + 1);
                }
            }
            best = __int_as_float(0xff800000);
            best_idx = -1;
            first_nan = false;
            return __shfl_sync(kFull, good, 0) != 0;
        };
        // Reduces the tile in `st` (nv vectors, the row's vectors v0..) into the running candidate; GT threads share it.
        auto reduce_tile = [&](auto group_threads, const uint4* st, int gt, int v0, int nv, bool row_start) {
            constexpr int GT = decltype(group_threads)::value;
            int bestq = -1;                                // vector (within this tile) of a new running maximum
#pragma unroll
            for (int i = 0; i < kBulkTileVec / GT; ++i) {
                const int q = gt + i * GT;
                if (q < nv) {
                    const uint4 v = st[q];
                    if (i == 0 && gt == 0 && row_start) first_nan = rm.v_offset == 0 && bf16_bits_nan(v.x & 0xFFFFu);
                    const float m = vec_max(v);
                    if (m > best) { best = m; bestq = q; }
                }
            }
            if (bestq >= 0) {                              // locate the element while the tile is still resident
                const uint4 v = st[bestq];
                best_idx = (v0 + bestq) * 8 + first_equal(v, best);
            }
        };
        auto ragged_tail = [&](int gt, long long row) {    // the row's last V mod 8 elements, by plain loads
            if (gt < ragged) {
                const int e = nvec_row * 8 + gt;
                const unsigned short b = __ldg(reinterpret_cast<const unsigned short*>(logits + actual_row(row) * stride) + e);
                const float x = __uint_as_float(static_cast<unsigned>(b) << 16);
                if (x > best) { best = x; best_idx = e; }
            }
        };

        if (plan.n_groups == 1) {
            // ---- large tiles: eight warps take every tile, one after the other
            if (warp < kWideGroupWarps) {
                constexpr int GT = kWideGroupWarps * 32;
                const int ct = threadIdx.x;
                int s = 0;
                uint32_t use = 0;
                for (int i = 0; i < n_rows && ok; ++i) {
                    const long long row = seq_row(i);
                    int tile, tile_hi;
                    tiles_of(row, tile, tile_hi);
                    for (; tile < tile_hi; ++tile) {
                        // the outcome of the wait is made uniform so that the warp leaves the loop together
                        if (!__all_sync(kFull, mbar_wait_bounded(&sh->full[s], use & 1u, abort))) { ok = false; break; }
                        const int v0 = tile * tile_vec;
                        const int nv = max(0, min(tile_vec, nvec_row - v0));
                        const uint4* st = reinterpret_cast<const uint4*>(stage_base + static_cast<size_t>(s) * plan.stage_bytes);
                        reduce_tile(std::integral_constant<int, GT>{}, st, ct, v0, nv, tile == 0);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&sh->empty[s]);
                        if (ragged != 0 && tile == tiles_per_row - 1) ragged_tail(ct, row);
                        if (++s == ns) { s = 0; ++use; }
                    }
                    if (ok && !hand_over(i)) ok = false;
                }
            }
        } else if (warp < n_cons) {
            // ---- small tiles: groups of four warps take the tiles in turn (tile number `it` of the CTA goes to group
            // it mod G and sits in stage it mod ns), so that what a tile costs beside its bytes overlaps between groups
            constexpr int GT = kSmallGroupWarps * 32, G = kSmallGroups;
            const int group = warp / kSmallGroupWarps;
            const int gt = threadIdx.x - group * GT;
            const int stage_bytes = plan.stage_bytes;
            long long cur_row = row_first;                 // rows before it have been handed over by this warp
            long long row = row_first;
            int tile = static_cast<int>(t0 - row * tiles_per_row) + group;
            while (tile >= tiles_per_row) { tile -= tiles_per_row; ++row; }
            const int n_tiles_cta = static_cast<int>(t1 - t0);
            int s = group % ns;                            // stage and use count of the group's next tile, kept incrementally:
            uint32_t use = static_cast<uint32_t>(group / ns);   // a division per tile would sit on the critical path
            const unsigned char* stage = stage_base + static_cast<size_t>(s) * stage_bytes;
            for (int it = group; it < n_tiles_cta && ok; it += G) {
                while (cur_row < row) {                    // rows finished (or never touched) by this group
                    if (!hand_over(static_cast<int>(cur_row - row_first))) { ok = false; break; }
                    ++cur_row;
                }
                if (!ok) break;
                if (!__all_sync(kFull, mbar_wait_bounded(&sh->full[s], use & 1u, abort))) { ok = false; break; }
                const int v0 = tile * tile_vec;
                const int nv = max(0, min(tile_vec, nvec_row - v0));
                reduce_tile(std::integral_constant<int, GT>{}, reinterpret_cast<const uint4*>(stage), gt, v0, nv, tile == 0);
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh->empty[s]);
                if (ragged != 0 && tile == tiles_per_row - 1) ragged_tail(gt, row);
                tile += G;
                while (tile >= tiles_per_row) { tile -= tiles_per_row; ++row; }
                s += G;                                    // G <= ns
                stage += static_cast<size_t>(G) * stage_bytes;
                if (s >= ns) { s -= ns; ++use; stage -= static_cast<size_t>(ns) * stage_bytes; }
            }
            // the rest of the CTA's rows (the last one this group worked on, and any behind it)
            while (ok && cur_row < row_first + n_rows) {
                ok = hand_over(static_cast<int>(cur_row - row_first));
                ++cur_row;
            }
        }
        if (!ok && lane == 0) {
            *abort = 1;
            atomicExch(status, kStatusWaitTimeout);
        }
        if (ft.mode != 0) serve_queue(sam, ft, epoch, sh, queue, abort, status, lane);
    }
    __syncthreads();
    if (ft.mode != 0 && threadIdx.x == 0) {
        // the CTA that leaves last has seen every other CTA read the launch count at its start: it moves the count on
        __threadfence();
        if (atomicAdd(ft.launch_words + 1, 1) == static_cast<int>(gridDim.x) - 1) {
            ft.launch_words[1] = 0;
            ft.launch_words[0] = epoch;
        }
    }
    if (sh->abort) {
        // copies already issued must land before this CTA's shared memory is given up
        if (threadIdx.x == 0) {
            const long long issued = sh->issued;
            const long long first = (issued > ns) ? issued - ns : 0;
            for (long long j = first; j < issued; ++j) {
                const int sj = static_cast<int>(j % ns);
                const uint32_t uj = static_cast<uint32_t>(j / ns);
                int never = 0;
                mbar_wait_bounded(&sh->full[sj], uj & 1u, &never);
            }
        }
        __syncthreads();
    }
}

}  // namespace samb200
