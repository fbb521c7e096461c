// Vocabulary argmax, bulk-copy pipelined variant (sm_100a). Included only by sam_capi.cu.
//
// One persistent CTA per SM.  A producer thread streams row tiles from HBM into a ring of
// shared-memory stages with 1-D bulk asynchronous copies (cp.async.bulk, completion counted on
// an mbarrier); the consumer warps reduce the tiles straight out of shared memory.  Loads cost
// no issue slots and no registers, ~190 KB per SM are in flight, and the reduction of one tile
// overlaps the copies of the following ones.  Requires 16-byte aligned rows (base and stride);
// the direct-load kernel covers everything else.
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
constexpr int kBulkThreads = kBulkConsumers + 32 + kBulkWalkerWarps * 32;   // consumers, producer warp, walkers
constexpr uint32_t kMaxPolls = 1u << 22;
constexpr size_t kBulkSmemBytes = static_cast<size_t>(kBulkStages) * kBulkTileBytes + 1024;

enum : int { kStatusOk = 0, kStatusWaitTimeout = 1 };

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
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
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
    long long issued;   // tiles the producer has issued copies for
    int abort;
};

__global__ void __launch_bounds__(kBulkThreads, 1)
argmax_bulk_kernel(const __nv_bfloat16* __restrict__ logits, long long stride, long long R, int V,
                   int tiles_per_row, int tile_vec, unsigned long long* __restrict__ keys,
                   int* __restrict__ status, DeviceSam sam, PreWalk pw) {
    // tile_vec <= kBulkTileVec: vectors per tile, chosen by the host so that a row splits into
    // tiles_per_row nearly equal tiles (large tiles amortise the per-tile hand-shake best).
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* stage_base = smem_raw;                                      // kBulkStages * 16 KB
    BulkShared* sh = reinterpret_cast<BulkShared*>(smem_raw + static_cast<size_t>(kBulkStages) * kBulkTileBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const long long total = R * tiles_per_row;
    const long long t0 = total * blockIdx.x / gridDim.x;
    const long long t1 = total * (blockIdx.x + 1) / gridDim.x;
    const int nvec_row = V >> 3;               // whole 16-byte vectors per row (rows are 16-byte aligned)
    const int ragged = V & 7;                  // trailing elements read with plain loads

    if (threadIdx.x == 0) {
        for (int s = 0; s < kBulkStages; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->empty[s], kBulkConsumerWarps);
        }
        sh->abort = 0;
        sh->issued = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    volatile int* abort = &sh->abort;

    if (warp == kBulkConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            long long it = 0;
            bool ok = true;
            long long row = t0 / tiles_per_row;
            int tile = static_cast<int>(t0 - row * tiles_per_row);
            int s = 0;
            uint32_t use = 0;
            for (long long t = t0; t < t1; ++t, ++it) {
                if (!mbar_wait_bounded(&sh->empty[s], (use & 1u) ^ 1u, abort)) { ok = false; break; }
                const int v0 = tile * tile_vec;
                const int nv = max(0, min(tile_vec, nvec_row - v0));
                if (nv > 0) {
                    const uint32_t bytes = static_cast<uint32_t>(nv) * 16u;
                    mbar_arrive_expect_tx(&sh->full[s], bytes);
                    bulk_load(stage_base + static_cast<size_t>(s) * kBulkTileBytes,
                              reinterpret_cast<const uint4*>(logits + row * stride) + v0, bytes, &sh->full[s]);
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
    } else if (warp > kBulkConsumerWarps) {
        // ------------------------------------------------------------------ walk-ahead warps
        if (pw.enabled) {
            const int w = warp - kBulkConsumerWarps - 1;
            for (int b = blockIdx.x * kBulkWalkerWarps + w; b < pw.B; b += gridDim.x * kBulkWalkerWarps)
                prewalk_stream(sam, pw, b, lane);
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int ct = threadIdx.x;                       // 0 .. kBulkConsumers-1
        long long cur_row = -1;
        float best = __int_as_float(0xff800000);          // -inf: only strictly greater values are candidates
        int best_idx = -1;
        bool ok = true;

        auto flush = [&]() {
            if (cur_row < 0) return;
            unsigned long long k = (best_idx >= 0) ? pack_candidate(best, static_cast<unsigned>(best_idx)) : 0ull;
            k = warp_max_u64(k);
            if (lane == 0 && k != 0ull) atomicMax(keys + cur_row, k);
        };

        long long row = t0 / tiles_per_row;
        int tile = static_cast<int>(t0 - row * tiles_per_row);
        int s = 0;
        uint32_t use = 0;
        for (long long t = t0; t < t1; ++t) {
            if (row != cur_row) {
                flush();
                cur_row = row;
                best = __int_as_float(0xff800000);
                best_idx = -1;
            }
            if (!mbar_wait_bounded(&sh->full[s], use & 1u, abort)) { ok = false; break; }
            const int v0 = tile * tile_vec;
            const int nv = max(0, min(tile_vec, nvec_row - v0));
            const uint4* st = reinterpret_cast<const uint4*>(stage_base + static_cast<size_t>(s) * kBulkTileBytes);
            int bestq = -1;                                // vector (within this tile) of a new running maximum
#pragma unroll
            for (int i = 0; i < kBulkTileVec / kBulkConsumers; ++i) {
                const int q = ct + i * kBulkConsumers;
                if (q < nv) {
                    const uint4 v = st[q];
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
                const unsigned short b = __ldg(reinterpret_cast<const unsigned short*>(logits + row * stride) + e);
                const float x = __uint_as_float(static_cast<unsigned>(b) << 16);
                if (x > best) { best = x; best_idx = e; }
            }
            if (++tile == tiles_per_row) { tile = 0; ++row; }
            if (++s == kBulkStages) { s = 0; ++use; }
        }
        if (ok) {
            flush();
        } else if (lane == 0) {
            *abort = 1;
            atomicExch(status, kStatusWaitTimeout);
        }
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
