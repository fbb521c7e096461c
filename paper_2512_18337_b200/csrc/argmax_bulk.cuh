// Vocabulary argmax, bulk-copy pipelined variant (sm_100a). Included only by sam_capi.cu.
//
// One persistent CTA per SM.  A producer thread streams row tiles from HBM into a ring of
// shared-memory stages with 1-D bulk asynchronous copies (cp.async.bulk, completion counted on
// an mbarrier); the consumer warps reduce the tiles straight out of shared memory.  Loads cost
// no issue slots and no registers, ~190 KB per SM are in flight, and the reduction of one tile
// overlaps the copies of the following ones.  Requires 16-byte aligned rows (base and stride);
// the direct-load kernel covers everything else.
//
// The consumer warps never touch global memory for their results: when a row (or the CTA's part of
// it) is finished, each warp leaves its candidate in a small ring in shared memory and moves on.
// A finisher warp combines the eight candidates of up to 32 rows at a time (one row per lane) and
// publishes them with one 64-bit atomic max per row, so that the round trips to L2 stay off the
// streaming path.
//
// Fused tail.  When the host asks for it, the accept step of a stream (decode the row results,
// longest matching prefix, follow the model's own token, next draft) runs inside this kernel as
// soon as the last partial result of the stream's K+1 rows has landed: after publishing a row the
// finisher adds the tiles this CTA reduced for it to a per-stream counter, the addition that
// completes the count puts the stream into a queue in the CTA's shared memory, and idle warps of
// that CTA (the walk-ahead warps, the finisher and the consumer warps once their work is done) take
// streams from the queue.  Nobody waits for another CTA, so the scheme needs no co-residency.
//
// Every wait on an mbarrier is bounded: after kMaxPolls unsuccessful polls the waiting thread
// raises the CTA's abort flag and the status word in global memory, all roles leave their
// loops, the producer waits (bounded again) for copies still in flight, and the CTA exits.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "sam_kernels.cuh"

namespace samb200 {

#ifndef SAM_BULK_TILE_VEC
#define SAM_BULK_TILE_VEC 4096
#endif
#ifndef SAM_BULK_STAGES
#define SAM_BULK_STAGES 3
#endif
#ifndef SAM_BULK_CONSUMER_WARPS
#define SAM_BULK_CONSUMER_WARPS 8
#endif
constexpr int kBulkTileVec = SAM_BULK_TILE_VEC;        // capacity of one stage in 16-byte vectors (64 KB)
constexpr int kBulkTileBytes = kBulkTileVec * 16;
constexpr int kBulkStages = SAM_BULK_STAGES;           // ring of kBulkStages * kBulkTileBytes (<= ~200 KB)
constexpr int kBulkConsumerWarps = SAM_BULK_CONSUMER_WARPS;
constexpr int kBulkConsumers = kBulkConsumerWarps * 32;
constexpr int kBulkWalkerWarps = 2;                    // spare warps that walk ahead along the drafts
constexpr int kBulkThreads = kBulkConsumers + 64 + kBulkWalkerWarps * 32;   // consumers, producer, finisher, walkers
constexpr int kRowSlots = 64;                          // ring of per-row candidate slots (consumers -> finisher)
constexpr uint32_t kMaxPolls = 1u << 22;
constexpr int kQueueCap = 1024;                        // streams one CTA can be handed (host checks the bound)
constexpr size_t kBulkCtrlOff = static_cast<size_t>(kBulkStages) * kBulkTileBytes;
constexpr size_t kBulkQueueOff = kBulkCtrlOff + 1024;
constexpr size_t kBulkCandOff = kBulkQueueOff + kQueueCap * 4;
constexpr size_t kBulkSmemBytes = kBulkCandOff + static_cast<size_t>(kRowSlots) * kBulkConsumerWarps * 8;

enum : int { kStatusOk = 0, kStatusWaitTimeout = 1, kStatusQueueOverflow = 2 };

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
    uint64_t full[kBulkStages];
    uint64_t empty[kBulkStages];
    long long issued;                 // tiles the producer has issued copies for
    int abort;
    int q_tail;                       // streams pushed into the queue
    int q_head;                       // tickets handed to worker warps
    int fin_rows;                     // rows of this CTA the finisher has published
    int fin_finished;                 // the finisher has left its loop: no pushes after that
    int prog[kBulkConsumerWarps];     // rows each consumer warp has handed over
};
static_assert(sizeof(BulkShared) <= 1024, "control block");

// Fused accept step (see the file header).  `done[b]` counts contributions to stream b and is
// zero between calls; `expected` is the count at which the stream is complete.
struct FusedTail {
    AcceptArgs args;
    int* done;       // [B]
    int expected;
    int mode;        // 0 = off, else kTailVerifyOnly + 1 or kTailResume + 1
};

__device__ __forceinline__ int ld_volatile_s32(const int* p) { return *reinterpret_cast<const volatile int*>(p); }
__device__ __forceinline__ void st_volatile_s32(int* p, int v) { *reinterpret_cast<volatile int*>(p) = v; }

__device__ __forceinline__ void fused_accept(const DeviceSam& sam, const FusedTail& ft, int b, int lane) {
    __threadfence();                 // order the reads below after the counter observation
    if (ft.mode == kTailResume + 1) accept_stream<kTailResume>(sam, ft.args, b, lane);
    else accept_stream<kTailVerifyOnly>(sam, ft.args, b, lane);
    if (lane == 0) ft.done[b] = 0;
}

// Idle warps serve the CTA's queue until the finisher has left its loop and the queue is drained.
// Each round takes one ticket; a ticket beyond the final tail means there is no more work.
__device__ __forceinline__ void serve_queue(const DeviceSam& sam, const FusedTail& ft, BulkShared* sh,
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
        fused_accept(sam, ft, b, lane);
    }
}

__global__ void __launch_bounds__(kBulkThreads, 1)
argmax_bulk_kernel(const __nv_bfloat16* __restrict__ logits, long long stride, long long R, int V,
                   int tiles_per_row, int tile_vec, unsigned long long* __restrict__ keys,
                   int* __restrict__ status, const __grid_constant__ DeviceSam sam,
                   const __grid_constant__ PreWalk pw, const __grid_constant__ FusedTail ft,
                   const __grid_constant__ RowMap rm) {
    // tile_vec <= kBulkTileVec: vectors per tile, chosen by the host so that a row splits into
    // tiles_per_row nearly equal tiles (large tiles amortise the per-tile hand-shake best).
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* stage_base = smem_raw;                                      // kBulkStages tiles
    BulkShared* sh = reinterpret_cast<BulkShared*>(smem_raw + kBulkCtrlOff);
    int* queue = reinterpret_cast<int*>(smem_raw + kBulkQueueOff);
    unsigned long long* cand = reinterpret_cast<unsigned long long*>(smem_raw + kBulkCandOff);   // [kRowSlots][warps]

    // the accept kernel may be scheduled now; it waits for this grid before it reads any result
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // with a row list the number of rows is only known on the device, and a CTA's share may be empty
    const long long n_all = (rm.list != nullptr) ? __ldg(rm.n_rows) : R;
    const long long total = n_all * tiles_per_row;
    const long long t0 = total * blockIdx.x / gridDim.x;
    const long long t1 = total * (blockIdx.x + 1) / gridDim.x;
    const long long row_first = t0 / tiles_per_row;      // position in the list (or the row itself without one)
    const int n_rows = (t1 > t0) ? static_cast<int>((t1 - 1) / tiles_per_row - row_first + 1) : 0;   // rows this CTA touches
    const int nvec_row = V >> 3;               // whole 16-byte vectors per row (rows are 16-byte aligned)
    const int ragged = V & 7;                  // trailing elements read with plain loads

    if (threadIdx.x == 0) {
        for (int s = 0; s < kBulkStages; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->empty[s], kBulkConsumerWarps);
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
    __syncthreads();
    volatile int* abort = &sh->abort;

    if (warp == kBulkConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            long long it = 0;
            bool ok = true;
            long long row = row_first;
            int tile = static_cast<int>(t0 - row * tiles_per_row);
            int s = 0;
            uint32_t use = 0;
            const uint64_t policy = l2_evict_first_policy();
            for (long long t = t0; t < t1; ++t, ++it) {
                // with a row list the row number is fetched before the wait, off the path of the copy
                const long long arow = (rm.list != nullptr) ? __ldg(rm.list + row) : row;
                if (!mbar_wait_bounded(&sh->empty[s], (use & 1u) ^ 1u, abort)) { ok = false; break; }
                const int v0 = tile * tile_vec;
                const int nv = max(0, min(tile_vec, nvec_row - v0));
                if (nv > 0) {
                    const uint32_t bytes = static_cast<uint32_t>(nv) * 16u;
                    mbar_arrive_expect_tx(&sh->full[s], bytes);
                    bulk_load(stage_base + static_cast<size_t>(s) * kBulkTileBytes,
                              reinterpret_cast<const uint4*>(logits + arow * stride) + v0, bytes, &sh->full[s], policy);
                } else {
                    mbar_arrive(&sh->full[s]);      // nothing to copy (row shorter than one vector)
                }
                if (++tile == tiles_per_row) { tile = 0; ++row; }
                if (++s == kBulkStages) { s = 0; ++use; }
            }
            sh->issued = it;
            if (!ok) {
                *abort = 1;
                atomicExch(status, kStatusWaitTimeout);
            }
        }
    } else if (warp == kBulkConsumerWarps + 1) {
        // ------------------------------------------------------------------ finisher
        const int K1 = ft.args.K + 1;
        int done_rows = 0;
        uint32_t polls = 0;
        while (done_rows < n_rows) {
            int p = (lane < kBulkConsumerWarps) ? ld_volatile_s32(&sh->prog[lane]) : 0x7fffffff;
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
                const long long row = (rm.list != nullptr) ? __ldg(rm.list + row_first + i) : row_first + i;
                const unsigned long long* c = cand + static_cast<size_t>(i % kRowSlots) * kBulkConsumerWarps;
                unsigned long long k = 0ull;
#pragma unroll
                for (int w = 0; w < kBulkConsumerWarps; ++w) {
                    const unsigned long long x = c[w];
                    k = (x > k) ? x : k;
                }
                if (k != 0ull) atomicMax(keys + row, k);
                if (ft.mode != 0) {
                    __threadfence();                   // the candidate first, then the count
                    const long long ra = row * tiles_per_row, rb = ra + tiles_per_row;
                    const int seg = static_cast<int>(min(rb, t1) - max(ra, t0));   // tiles of the row this CTA reduced
                    const int b = static_cast<int>(row / K1);
                    if (atomicAdd(ft.done + b, seg) + seg == ft.expected) {
                        __threadfence();
                        const int slot = atomicAdd(&sh->q_tail, 1);
                        if (slot < kQueueCap) st_volatile_s32(queue + slot, b);
                        else atomicExch(status, kStatusQueueOverflow);   // the host sizes the grid so that this cannot happen
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
            serve_queue(sam, ft, sh, queue, abort, status, lane);
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
                        last = (atomicAdd(ft.done + b, 1) + 1 == ft.expected);
                    }
                    __syncwarp();
                    if (__shfl_sync(kFull, last, 0)) fused_accept(sam, ft, b, lane);
                }
            }
        }
        if (ft.mode != 0) serve_queue(sam, ft, sh, queue, abort, status, lane);
    } else {
        // ------------------------------------------------------------------ consumers
        const int ct = threadIdx.x;                       // 0 .. kBulkConsumers-1
        long long cur_row = -1;
        float best = __int_as_float(0xff800000);          // -inf: only strictly greater values are candidates
        int best_idx = -1;
        bool first_nan = false;                           // element 0 of the current row is NaN (seen by thread 0 only)
        bool ok = true;

        // Hands the finished row over to the finisher: candidate into the row's slot, then the progress counter.
        auto flush = [&]() -> bool {
            if (cur_row < 0) return true;
            unsigned long long k = (best_idx >= 0) ? pack_candidate(best, static_cast<unsigned>(best_idx + rm.v_offset)) : 0ull;
            if (first_nan) k = kCandidateFirstIsNaN;
            k = warp_max_u64(k);
            int good = 1;
            if (lane == 0) {
                const int i = static_cast<int>(cur_row - row_first);
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
            return __shfl_sync(kFull, good, 0) != 0;
        };

        long long row = row_first;
        int tile = static_cast<int>(t0 - row * tiles_per_row);
        int s = 0;
        uint32_t use = 0;
        for (long long t = t0; t < t1; ++t) {
            if (row != cur_row) {
                if (!flush()) { ok = false; break; }
                cur_row = row;
                best = __int_as_float(0xff800000);
                best_idx = -1;
                first_nan = false;
            }
            // the outcome of the wait is made uniform so that the warp leaves the loop together
            if (!__all_sync(kFull, mbar_wait_bounded(&sh->full[s], use & 1u, abort))) { ok = false; break; }
            const int v0 = tile * tile_vec;
            const int nv = max(0, min(tile_vec, nvec_row - v0));
            const uint4* st = reinterpret_cast<const uint4*>(stage_base + static_cast<size_t>(s) * kBulkTileBytes);
            int bestq = -1;                                // vector (within this tile) of a new running maximum
#pragma unroll
            for (int i = 0; i < kBulkTileVec / kBulkConsumers; ++i) {
                const int q = ct + i * kBulkConsumers;
                if (q < nv) {
                    const uint4 v = st[q];
                    if (i == 0 && ct == 0 && tile == 0) first_nan = rm.v_offset == 0 && bf16_bits_nan(v.x & 0xFFFFu);
                    const float m = vec_max(v);
                    if (m > best) { best = m; bestq = q; }
                }
            }
            if (bestq >= 0) {                              // locate the element while the tile is still resident
                const uint4 v = st[bestq];
                best_idx = (v0 + bestq) * 8 + first_equal(v, best);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->empty[s]);
            if (ragged != 0 && tile == tiles_per_row - 1 && ct < ragged) {
                const int e = nvec_row * 8 + ct;
                const long long arow = (rm.list != nullptr) ? __ldg(rm.list + row) : row;
                const unsigned short b = __ldg(reinterpret_cast<const unsigned short*>(logits + arow * stride) + e);
                const float x = __uint_as_float(static_cast<unsigned>(b) << 16);
                if (e == 0) first_nan = rm.v_offset == 0 && bf16_bits_nan(b);   // rows shorter than one vector
                if (x > best) { best = x; best_idx = e; }
            }
            if (++tile == tiles_per_row) { tile = 0; ++row; }
            if (++s == kBulkStages) { s = 0; ++use; }
        }
        if (ok) ok = flush();
        if (!ok && lane == 0) {
            *abort = 1;
            atomicExch(status, kStatusWaitTimeout);
        }
        if (ft.mode != 0) serve_queue(sam, ft, sh, queue, abort, status, lane);
    }
    __syncthreads();
    if (sh->abort) {
        // copies already issued must land before this CTA's shared memory is given up
        if (threadIdx.x == 0) {
            const long long issued = sh->issued;
            const long long first = (issued > kBulkStages) ? issued - kBulkStages : 0;
            for (long long j = first; j < issued; ++j) {
                const int sj = static_cast<int>(j % kBulkStages);
                const uint32_t uj = static_cast<uint32_t>(j / kBulkStages);
                int never = 0;
                mbar_wait_bounded(&sh->full[sj], uj & 1u, &never);
            }
        }
        __syncthreads();
    }
}

}  // namespace samb200
