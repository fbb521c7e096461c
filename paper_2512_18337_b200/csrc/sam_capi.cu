// C ABI of the library: argument checks, device-blob upload and kernel launches.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstdlib>
#include <atomic>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "sam.h"
#include "sam_index.h"
#include "sam_kernels.cuh"
#include "argmax_bulk.cuh"
#include "sam_update.cuh"

using namespace samb200;

namespace {

thread_local int g_last_cuda = 0;
std::atomic<long long> g_launches{0};   // kernels this library has enqueued (diagnostic)

inline int cuda_fail(cudaError_t e) {
    g_last_cuda = static_cast<int>(e);
    return SAM_ERR_CUDA;
}

#define SAM_CUDA(call)                                   \
    do {                                                 \
        cudaError_t e__ = (call);                        \
        if (e__ != cudaSuccess) return cuda_fail(e__);   \
    } while (0)

struct DeviceInfo {
    int sms = 0;
};

int device_info(DeviceInfo* out) {
    static thread_local int cached_dev = -1;
    static thread_local DeviceInfo cached;
    int dev = 0;
    SAM_CUDA(cudaGetDevice(&dev));
    if (dev != cached_dev) {
        int sms = 0;
        SAM_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        cached.sms = sms;
        cached_dev = dev;
    }
    *out = cached;
    return SAM_OK;
}

// ---- optional per-kernel timing (events owned by the library) --------------------------------
struct Profile {
    std::vector<cudaEvent_t> ev;   // 3 per call
    int32_t cap = 0, used = 0;
};
Profile g_prof;

inline void prof_mark(int phase, cudaStream_t st) {
    if (g_prof.used < g_prof.cap) cudaEventRecord(g_prof.ev[static_cast<size_t>(g_prof.used) * 3 + phase], st);
}
inline void prof_done() {
    if (g_prof.used < g_prof.cap) ++g_prof.used;
}

inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int check_verify_args(const void* logits, int64_t stride, int32_t B, int32_t K, int32_t V,
                      const int32_t* drafts, const int32_t* n_draft, int32_t* argmax_out,
                      int32_t* accepted, int32_t* n_accepted, void* ws, int64_t ws_bytes) {
    if (B < 0 || K < 1 || K > SAM_K_MAX || V < 1 || stride < V) return SAM_ERR_INVALID_ARG;
    if (B == 0) return SAM_OK;
    if (!logits || !drafts || !n_draft || !argmax_out || !accepted || !n_accepted || !ws) return SAM_ERR_INVALID_ARG;
    if (!aligned(logits, 2) || !aligned(ws, 8)) return SAM_ERR_INVALID_ARG;
    if (ws_bytes < sam_workspace_bytes(B, K)) return SAM_ERR_TOO_SMALL;
    return SAM_OK;
}

int g_argmax_variant = 0;   // 0 = by alignment and size, 1 = direct loads always, 2 = bulk-copy (if aligned) with the accept step inside, 3 = bulk-copy (if aligned) + accept kernel

inline int* status_word(unsigned long long* keys, int64_t R) {
    return reinterpret_cast<int*>(reinterpret_cast<char*>(keys) + ((R * 8 + 255) / 256) * 256);
}

// Partial results land in keys[R]; `status` receives a non-zero code if a kernel gives up on an
// internal wait.
// Layout of the verification scratch:
// keys[R] | status (256 B) | pre_state[B*K] | pre_len[B*K] | done[B] | row_list[R] | list meta words (256 B) | rowcnt[R] | acc_epoch[B]
struct Scratch {
    unsigned long long* keys;
    int* status;
    int* pre_state;
    int* pre_len;
    int* done;
    int* row_list;
    int* list_meta;
    int* rowcnt;
    int* acc_epoch;
    int64_t bytes;
};
Scratch scratch_layout(void* base, int32_t B, int32_t K, int32_t M = 1) {   // M: automaton slots per stream (walk-ahead arrays)
    auto up = [](int64_t x) { return (x + 255) & ~int64_t(255); };
    const int64_t R = static_cast<int64_t>(B) * (K + 1);
    char* p = static_cast<char*>(base);
    Scratch s;
    int64_t o = 0;
    s.keys = reinterpret_cast<unsigned long long*>(p + o);  o = up(o + R * 8);
    s.status = reinterpret_cast<int*>(p + o);               o += 256;
    s.pre_state = reinterpret_cast<int*>(p + o);            o = up(o + static_cast<int64_t>(B) * M * K * 4);
    s.pre_len = reinterpret_cast<int*>(p + o);              o = up(o + static_cast<int64_t>(B) * M * K * 4);
    s.done = reinterpret_cast<int*>(p + o);                 o = up(o + static_cast<int64_t>(B) * 4);
    s.row_list = reinterpret_cast<int*>(p + o);             o = up(o + R * 4);
    s.list_meta = reinterpret_cast<int*>(p + o);            o += 256;
    s.rowcnt = reinterpret_cast<int*>(p + o);               o = up(o + R * 4);
    s.acc_epoch = reinterpret_cast<int*>(p + o);            o = up(o + static_cast<int64_t>(B) * 4);
    s.bytes = o;
    return s;
}

// Enqueues the argmax over R rows.  With the bulk-copy kernel two more things can ride along:
// the walk-ahead over the drafts (pw) and the accept step of every stream (tail; needs `done`).
// *did_prewalk / *did_tail tell the caller what the launch will have done; whatever it did not do
// is left to a separate accept kernel.
int launch_argmax(const void* logits, int64_t stride, int64_t R, int32_t V, unsigned long long* keys,
                  int* status, cudaStream_t st, const DeviceSam* sam = nullptr, const PreWalk* pw = nullptr,
                  bool* did_prewalk = nullptr, const AcceptArgs* tail = nullptr, int tail_mode = 0,
                  int* done = nullptr, bool* did_tail = nullptr, const RowMap* rmap = nullptr, int* rowcnt = nullptr,
                  int* acc_epoch = nullptr, int* launch_words = nullptr) {
    // Below about 0.8 GB of logits the direct-load kernel followed by an accept kernel that walks the proposal before its
    // grid-dependency wait is the faster pair: it starts sooner than the bulk-copy pipeline and finishes more evenly
    // (measured per step, direct vs bulk-copy: 11.4 vs 13.4 us at B = 4, K = 3; 11.7 vs 13.8 us on the tiny workload;
    // 39.2 vs 40.9 us at 175 MB; 105.9 vs 107.1 us at 660 MB; 153.2 vs 151.2 us at 990 MB; 197.1 vs 195.3 us at 1.3 GB).
    // Proposals longer than 16 tokens stay with the bulk-copy kernel at every size: their walk-ahead is long and its
    // spare warps hide it better (K = 32: 45.6 vs 38.2 us at 160 MB).
    const bool latency_case = g_argmax_variant == 0 && tail != nullptr && tail->K <= 16 &&
                              R * static_cast<int64_t>(V) * 2 <= (int64_t(768) << 20);
    prof_mark(0, st);
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != SAM_OK) return rc;
    const bool rows_aligned = aligned(logits, 16) && (stride % 8) == 0 && V >= 8;
    const bool bulk = rows_aligned && g_argmax_variant != 1 && !latency_case;
    const RowMap rm = rmap ? *rmap : RowMap{nullptr, nullptr, 0, 0, nullptr};
    if (did_prewalk) *did_prewalk = false;
    if (did_tail) *did_tail = false;
    if (bulk) {
        static thread_local int attr_dev = -1;
        int dev = 0;
        SAM_CUDA(cudaGetDevice(&dev));
        if (attr_dev != dev) {
            SAM_CUDA(cudaFuncSetAttribute(argmax_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(kBulkSmemBytes)));
            attr_dev = dev;
        }
        // a row is cut into the fewest tiles that fit a stage, all nearly equal (large tiles amortise what a tile costs
        // beside its bytes); the R * tiles_per_row tiles are split into equal contiguous ranges, one persistent CTA per SM
        const BulkPlan plan = bulk_plan(V);
        const int tiles_per_row = plan.tiles_per_row;
        const int64_t total = R * tiles_per_row;
        int64_t grid = di.sms;
        if (grid > total) grid = total;
        if (grid < 1) grid = 1;
        const bool prewalk = pw != nullptr && pw->enabled != 0;
        FusedTail ft{};
        if (tail != nullptr && done != nullptr && rowcnt != nullptr && acc_epoch != nullptr && launch_words != nullptr &&
            g_argmax_variant == 2 &&
            rm.list == nullptr && plan.n_groups == 1) {
            // a CTA is handed at most the streams that overlap its contiguous range of rows; it takes the used rows of
            // that range first, which it can do for up to kOrderCap rows of up to 32 streams
            const int64_t rows_per_cta = (total + grid - 1) / grid / tiles_per_row + 2;
            const int64_t streams_per_cta = rows_per_cta / (tail->K + 1) + 2;
            if (rows_per_cta <= kOrderCap && streams_per_cta <= 32) {
                ft.args = *tail;
                ft.args.flags |= kLeaveUnusedRows;
                ft.args.acc_epoch = acc_epoch;
                ft.launch_words = launch_words;
                ft.done = done;
                ft.rowcnt = rowcnt;
                ft.prewalk = prewalk ? 1 : 0;
                ft.mode = tail_mode + 1;
            }
        }
        argmax_bulk_kernel<<<static_cast<unsigned>(grid), kBulkThreads, kBulkSmemBytes, st>>>(
            static_cast<const __nv_bfloat16*>(logits), stride, R, V, plan, keys, status,
            sam ? *sam : DeviceSam{}, pw ? *pw : PreWalk{}, ft, rm);
        ++g_launches;
        if (did_prewalk) *did_prewalk = prewalk;
        if (did_tail) *did_tail = ft.mode != 0;
    } else {
        const int64_t nvec_max = (static_cast<int64_t>(V) + 7 + 7) / 8;   // worst-case leading offset of 7 elements
        const int tiles_per_row = static_cast<int>((nvec_max + kTileVec - 1) / kTileVec);
        const int64_t total = R * tiles_per_row;
        int64_t grid = static_cast<int64_t>(di.sms) * kDirectCtasPerSm;
        if (grid > total) grid = total;
        if (grid < 1) grid = 1;
        argmax_direct_kernel<<<static_cast<unsigned>(grid), kArgmaxThreads, 0, st>>>(
            static_cast<const __nv_bfloat16*>(logits), stride, R, V, tiles_per_row, keys, rm);
        ++g_launches;
    }
    SAM_CUDA(cudaGetLastError());
    prof_mark(1, st);
    return SAM_OK;
}

template <int kMode>
int launch_accept(const DeviceSam& sam, const AcceptArgs& a, cudaStream_t st, bool after_own_argmax = true) {
    const int warps = 4;
    const unsigned grid = static_cast<unsigned>((a.B + warps - 1) / warps);
    if (!after_own_argmax) {
        // whatever precedes in the stream may still be producing this kernel's inputs: ordinary stream order
        accept_kernel<kMode, false><<<grid, warps * 32, 0, st>>>(sam, a);
        SAM_CUDA(cudaGetLastError());
        ++g_launches;
        return SAM_OK;
    }
    // launched as a programmatic dependent of the kernel before it in the stream (the argmax kernel): its
    // blocks are placed, and load what does not depend on that kernel, while that kernel is still running
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    SAM_CUDA(cudaLaunchKernelEx(&cfg, accept_kernel<kMode, true>, sam, a));
    ++g_launches;
    return SAM_OK;
}

// ---- growing index: device side of an update ---------------------------------------------------
void set_device_view(sam_index* idx, void* device_buf) {
    const DeviceLayout& L = idx->layout;
    char* base = static_cast<char*>(device_buf);
    DeviceSam& d = idx->dev;
    d.rec = reinterpret_cast<const StateRec*>(base + L.rec_off);
    d.wide = reinterpret_cast<const Edge*>(base + L.edge_off);
    d.root_dst = reinterpret_cast<const int32_t*>(base + L.root_off);
    d.corpus = reinterpret_cast<const int32_t*>(base + L.corpus_off);
    d.root_span = static_cast<int32_t>(L.root_span);
    d.n_sep = static_cast<int32_t>(idx->seps.size());
    for (int k = 0; k < SAM_MAX_SEPARATORS; ++k) d.seps[k] = (k < d.n_sep) ? idx->seps[k] : -1;
}

// Copies a whole image (first upload, or after the wide rows were laid out afresh).
int apply_full(sam_index* idx, const Delta& D, cudaStream_t st) {
    const DeviceLayout& L = idx->layout;
    char* base = static_cast<char*>(idx->device_buf);
    SAM_CUDA(cudaMemcpyAsync(base + L.rec_off, D.all_rec.data(), D.all_rec.size() * sizeof(StateRec), cudaMemcpyHostToDevice, st));
    if (!D.all_wide.empty())
        SAM_CUDA(cudaMemcpyAsync(base + L.edge_off, D.all_wide.data(), D.all_wide.size() * sizeof(Edge), cudaMemcpyHostToDevice, st));
    SAM_CUDA(cudaMemcpyAsync(base + L.root_off, D.all_root.data(), D.all_root.size() * 4, cudaMemcpyHostToDevice, st));
    if (!D.all_corpus.empty())
        SAM_CUDA(cudaMemcpyAsync(base + L.corpus_off, D.all_corpus.data(), D.all_corpus.size() * 4, cudaMemcpyHostToDevice, st));
    return SAM_OK;
}

}  // namespace

// ---- small updates sent ahead of time -------------------------------------------------------------
// The builder thread copies every small update into a slot of the blob's ring as soon as it is packed: through
// page-locked memory, on a stream of the library's own, while decoding steps run on the caller's stream.  The copy
// touches nothing that a kernel reads.  sam_sync then only makes the caller's stream wait for the slot's event
// and launches the one kernel that scatters the slot into the live records - the only work that has to sit between
// two steps.  A slot is reused once the kernel that read it has finished.
struct samb200::UpdateRing {
    int device = -1;
    cudaStream_t copy_stream = nullptr;
    char* pinned = nullptr;                       // kRingSlots * kRingSlotBytes, page-locked
    char* dev_ring = nullptr;                     // the ring inside the caller's blob
    cudaEvent_t copied[kRingSlots] = {};          // the slot's copy has arrived
    cudaEvent_t applied[kRingSlots] = {};         // the kernel that read the slot has finished
    enum : int { kFree = 0, kStaged = 1, kApplied = 2 };
    int state[kRingSlots] = {};
    int next = 0;
    uint64_t epoch = 0;                           // changes with every (re-)upload: slots staged before it are void
    bool enabled = false;
    std::mutex mu;
};

namespace {

void ring_destroy(sam_index* idx) {
    UpdateRing* r = idx->ring;
    if (!r) return;
    int prev = -1;
    cudaGetDevice(&prev);
    if (r->device >= 0) cudaSetDevice(r->device);
    if (r->copy_stream) {
        cudaStreamSynchronize(r->copy_stream);
        cudaStreamDestroy(r->copy_stream);
    }
    for (int k = 0; k < kRingSlots; ++k) {
        if (r->copied[k]) cudaEventDestroy(r->copied[k]);
        if (r->applied[k]) { cudaEventSynchronize(r->applied[k]); cudaEventDestroy(r->applied[k]); }
    }
    if (r->pinned) cudaFreeHost(r->pinned);
    if (prev >= 0) cudaSetDevice(prev);
    delete r;
    idx->ring = nullptr;
}

// (Re-)creates the ring for the blob just uploaded; everything staged for an earlier blob is void.  Setup, not hot path.
int ring_attach(sam_index* idx, char* dev_ring) {
    UpdateRing* r = idx->ring;
    if (!r) {
        r = new (std::nothrow) UpdateRing();
        if (!r) return SAM_ERR_NOMEM;
        idx->ring = r;
    }
    std::lock_guard<std::mutex> lock(r->mu);
    r->enabled = false;
    int dev = 0;
    SAM_CUDA(cudaGetDevice(&dev));
    if (r->copy_stream && r->device != dev) return SAM_ERR_INVALID_ARG;      // a handle stays on the device of its first upload
    r->device = dev;
    if (!r->copy_stream) {
        SAM_CUDA(cudaStreamCreateWithFlags(&r->copy_stream, cudaStreamNonBlocking));
        void* hp = nullptr;
        SAM_CUDA(cudaHostAlloc(&hp, static_cast<size_t>(kRingSlots * kRingSlotBytes), cudaHostAllocDefault));
        r->pinned = static_cast<char*>(hp);
        for (int k = 0; k < kRingSlots; ++k) {
            SAM_CUDA(cudaEventCreateWithFlags(&r->copied[k], cudaEventDisableTiming));
            SAM_CUDA(cudaEventCreateWithFlags(&r->applied[k], cudaEventDisableTiming));
        }
    } else {
        SAM_CUDA(cudaStreamSynchronize(r->copy_stream));
    }
    for (int k = 0; k < kRingSlots; ++k) r->state[k] = UpdateRing::kFree;
    r->next = 0;
    ++r->epoch;
    r->dev_ring = dev_ring;
    r->enabled = true;
    return SAM_OK;
}

}  // namespace

// Builder thread: the update goes to the next ring slot if it is small enough and a slot is free; otherwise it stays
// as it is and sam_sync copies it on the caller's stream.
void samb200::ring_stage_async(sam_index* idx, Delta* D) {
    UpdateRing* r = idx->ring;
    if (!r || D->full || D->status != SAM_OK) return;
    StagedLayout L;
    staged_layout(*D, &L);
    if (L.total <= 0 || L.total > kRingSlotBytes) return;
    int k = -1, was = 0;
    uint64_t epoch = 0;
    {
        std::lock_guard<std::mutex> lock(r->mu);
        if (!r->enabled || r->state[r->next] == UpdateRing::kStaged) return;     // no blob yet, or sam_sync is 8 updates behind
        k = r->next;
        was = r->state[k];
        r->state[k] = UpdateRing::kStaged;
        r->next = (k + 1) % kRingSlots;
        epoch = r->epoch;
    }
    static thread_local int dev_set = -1;
    bool ok = true;
    if (dev_set != r->device) {
        ok = cudaSetDevice(r->device) == cudaSuccess;
        if (ok) dev_set = r->device;
    }
    // the kernel that read this slot last (and with it the copy that filled it) must be over
    if (ok && was == UpdateRing::kApplied) ok = cudaEventSynchronize(r->applied[k]) == cudaSuccess;
    if (ok) {
        char* h = r->pinned + k * kRingSlotBytes;
        staged_fill(*D, L, h);
        ok = cudaMemcpyAsync(r->dev_ring + k * kRingSlotBytes, h, static_cast<size_t>(L.total), cudaMemcpyHostToDevice,
                             r->copy_stream) == cudaSuccess &&
             cudaEventRecord(r->copied[k], r->copy_stream) == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        std::lock_guard<std::mutex> lock(r->mu);
        if (r->epoch == epoch) r->state[k] = UpdateRing::kFree;
        return;
    }
    D->staged_slot = k;
    D->staged_epoch = epoch;
    D->staged = L;
}

namespace {

UpdateArgs update_args(sam_index* idx, const Delta& D, const StagedLayout& L, const char* stage) {
    const DeviceLayout& dl = idx->layout;
    char* base = static_cast<char*>(idx->device_buf);
    UpdateArgs a{};
    a.rec = reinterpret_cast<StateRec*>(base + dl.rec_off);
    a.wide = reinterpret_cast<Edge*>(base + dl.edge_off);
    a.root = reinterpret_cast<int32_t*>(base + dl.root_off);
    a.corpus = reinterpret_cast<int32_t*>(base + dl.corpus_off) + D.corpus_off;
    a.stage = stage;
    a.off_ids = L.off_ids; a.off_recs = L.off_recs; a.off_descs = L.off_descs; a.off_edges = L.off_edges;
    a.off_rtok = L.off_rtok; a.off_rdst = L.off_rdst; a.off_tail = L.off_tail;
    a.n_rec = L.n_rec; a.n_seg = L.n_seg; a.n_root = L.n_root; a.n_tail = L.n_tail;
    a.root_span = static_cast<int>(dl.root_span);
    return a;
}

// The stream states to repair after an update (sam_sync_renormalize), or nothing (B = 0).
struct Renorm {
    int32_t B = 0;
    int32_t* state = nullptr;
    const int32_t* matched_len = nullptr;
};

// Launches the scatter kernel over a staged buffer; with `rn`, the kernel also repairs the stream states at its end.
int launch_update_kernel(sam_index* idx, const Delta& D, const StagedLayout& L, const char* stage, const Renorm* rn,
                         cudaStream_t st) {
    const UpdateArgs a = update_args(idx, D, L, stage);
    RenormTail t{};
    if (rn && rn->B > 0) {
        t.sam = idx->dev;
        t.sam.n_states = static_cast<int32_t>(D.n_states_after);       // the view this update leaves behind
        t.sam.n_corpus = D.n_tokens_after;
        t.B = rn->B;
        t.state = rn->state;
        t.matched_len = rn->matched_len;
        t.blocks_done = reinterpret_cast<unsigned*>(static_cast<char*>(idx->device_buf) + idx->layout.ctrl_off);
    }
    const int64_t work = std::max(std::max<int64_t>(L.n_rec, int64_t(L.n_seg) * 32), std::max<int64_t>(L.n_root, L.n_tail));
    const unsigned blocks = static_cast<unsigned>(std::min<int64_t>(1184, std::max<int64_t>(1, (work + 255) / 256)));
    apply_update_kernel<<<blocks, 256, 0, st>>>(a, t);
    SAM_CUDA(cudaGetLastError());
    ++g_launches;
    return SAM_OK;
}

int copy_long_rows(sam_index* idx, const Delta& D, cudaStream_t st) {
    Edge* wide = reinterpret_cast<Edge*>(static_cast<char*>(idx->device_buf) + idx->layout.edge_off);
    for (const WideSeg& g : D.segs)
        if (g.len >= kDirectRowEdges)
            SAM_CUDA(cudaMemcpyAsync(wide + g.dst_off, D.seg_edges.data() + g.src_off,
                                     static_cast<size_t>(g.len) * sizeof(Edge), cudaMemcpyHostToDevice, st));
    return SAM_OK;
}

bool has_long_rows(const Delta& D) {
    for (const WideSeg& g : D.segs)
        if (g.len >= kDirectRowEdges) return true;
    return false;
}

// Scatters one update.  *renormalized tells whether the launch also repaired the stream states of `rn`.
// Host buffers are pageable, so every cudaMemcpyAsync has taken its copy of the source when it returns.
int apply_changes(sam_index* idx, const Delta& D, cudaStream_t st, const Renorm* rn, bool* renormalized) {
    const DeviceLayout& L = idx->layout;
    char* base = static_cast<char*>(idx->device_buf);
    char* stage = base + L.stage_off;
    StateRec* rec = reinterpret_cast<StateRec*>(base + L.rec_off);
    Edge* wide = reinterpret_cast<Edge*>(base + L.edge_off);
    int32_t* root = reinterpret_cast<int32_t*>(base + L.root_off);
    const int64_t n_rec = static_cast<int64_t>(D.rec_ids.size());
    *renormalized = false;
    // rows long enough to be copied on their own must be in place before the states are repaired
    const Renorm* tail = (rn && rn->B > 0 && !has_long_rows(D)) ? rn : nullptr;
    // ---- already on the device: the builder thread sent it to a ring slot
    UpdateRing* r = idx->ring;
    if (D.staged_slot >= 0 && r) {
        bool valid;
        {
            std::lock_guard<std::mutex> lock(r->mu);
            valid = r->enabled && r->epoch == D.staged_epoch;
        }
        if (valid) {
            const int k = D.staged_slot;
            // normally the copy arrived long ago; only if it has not does the caller's stream have to wait for it
            if (cudaEventQuery(r->copied[k]) != cudaSuccess) {
                cudaGetLastError();
                SAM_CUDA(cudaStreamWaitEvent(st, r->copied[k], 0));
            }
            int rc = launch_update_kernel(idx, D, D.staged, r->dev_ring + k * kRingSlotBytes, tail, st);
            if (rc != SAM_OK) return rc;
            SAM_CUDA(cudaEventRecord(r->applied[k], st));
            {
                std::lock_guard<std::mutex> lock(r->mu);
                if (r->epoch == D.staged_epoch) r->state[k] = UpdateRing::kApplied;
            }
            *renormalized = tail != nullptr;
            return copy_long_rows(idx, D, st);
        }
    }
    // ---- small update that was not sent ahead: one page-locked buffer, one copy and one kernel on the caller's stream
    {
        StagedLayout a;
        staged_layout(D, &a);
        if (a.total <= kRingSlotBytes && a.total <= L.stage_bytes) {
            if (!idx->pinned_stage) {
                void* hp = nullptr;
                cudaEvent_t ev = nullptr;
                SAM_CUDA(cudaHostAlloc(&hp, static_cast<size_t>(kRingSlotBytes), cudaHostAllocDefault));
                const cudaError_t e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
                if (e != cudaSuccess) { cudaFreeHost(hp); return cuda_fail(e); }
                idx->pinned_stage = hp;
                idx->pinned_bytes = kRingSlotBytes;
                idx->stage_event = ev;
            } else {
                // the previous update's copy must have left the buffer before it is refilled
                SAM_CUDA(cudaEventSynchronize(static_cast<cudaEvent_t>(idx->stage_event)));
            }
            char* h = static_cast<char*>(idx->pinned_stage);
            staged_fill(D, a, h);
            if (a.total > 0) {
                SAM_CUDA(cudaMemcpyAsync(stage, h, static_cast<size_t>(a.total), cudaMemcpyHostToDevice, st));
                SAM_CUDA(cudaEventRecord(static_cast<cudaEvent_t>(idx->stage_event), st));
                const int rc = launch_update_kernel(idx, D, a, stage, tail, st);
                if (rc != SAM_OK) return rc;
                *renormalized = tail != nullptr;
            }
            return copy_long_rows(idx, D, st);
        }
    }
    // ---- large update: section by section through the staging area
    std::vector<char> buf;
    // records: [ids (padded to 32 B)] [records]
    const int64_t per_round = (L.stage_bytes - 64) / 36;
    for (int64_t i0 = 0; i0 < n_rec; i0 += per_round) {
        const int64_t n = std::min(per_round, n_rec - i0);
        const int64_t ids_bytes = (n * 4 + 31) & ~int64_t(31);
        buf.resize(static_cast<size_t>(ids_bytes + n * 32));
        std::memcpy(buf.data(), D.rec_ids.data() + i0, static_cast<size_t>(n) * 4);
        std::memcpy(buf.data() + ids_bytes, D.recs.data() + i0, static_cast<size_t>(n) * 32);
        SAM_CUDA(cudaMemcpyAsync(stage, buf.data(), buf.size(), cudaMemcpyHostToDevice, st));
        scatter_records_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(
            rec, reinterpret_cast<const int32_t*>(stage), reinterpret_cast<const StateRec*>(stage + ids_bytes),
            static_cast<int>(n));
        SAM_CUDA(cudaGetLastError());
        ++g_launches;
    }
    // wide rows: long ones directly, short ones in batches of [descriptors] [edges]
    std::vector<SegDesc> descs;
    std::vector<Edge> edges;
    auto flush_rows = [&]() -> int {
        if (descs.empty()) return SAM_OK;
        const int64_t d_bytes = (static_cast<int64_t>(descs.size()) * sizeof(SegDesc) + 31) & ~int64_t(31);
        buf.resize(static_cast<size_t>(d_bytes) + edges.size() * sizeof(Edge));
        std::memcpy(buf.data(), descs.data(), descs.size() * sizeof(SegDesc));
        std::memcpy(buf.data() + d_bytes, edges.data(), edges.size() * sizeof(Edge));
        SAM_CUDA(cudaMemcpyAsync(stage, buf.data(), buf.size(), cudaMemcpyHostToDevice, st));
        const int n = static_cast<int>(descs.size());
        copy_rows_kernel<<<static_cast<unsigned>((n + 7) / 8), 256, 0, st>>>(
            wide, reinterpret_cast<const SegDesc*>(stage), reinterpret_cast<const Edge*>(stage + d_bytes), n);
        SAM_CUDA(cudaGetLastError());
        ++g_launches;
        descs.clear();
        edges.clear();
        return SAM_OK;
    };
    for (const WideSeg& g : D.segs) {
        if (g.len >= kDirectRowEdges) {
            SAM_CUDA(cudaMemcpyAsync(wide + g.dst_off, D.seg_edges.data() + g.src_off, static_cast<size_t>(g.len) * sizeof(Edge),
                                     cudaMemcpyHostToDevice, st));
            continue;
        }
        const int64_t need = (static_cast<int64_t>(descs.size()) + 1) * sizeof(SegDesc) + 32 +
                             (static_cast<int64_t>(edges.size()) + g.len) * sizeof(Edge);
        if (need > L.stage_bytes) {
            const int rc = flush_rows();
            if (rc != SAM_OK) return rc;
        }
        descs.push_back(SegDesc{g.dst_off, static_cast<int>(edges.size()), g.len});
        edges.insert(edges.end(), D.seg_edges.begin() + g.src_off, D.seg_edges.begin() + g.src_off + g.len);
    }
    {
        const int rc = flush_rows();
        if (rc != SAM_OK) return rc;
    }
    // root entries: [tokens (padded)] [destinations]
    const int64_t n_root = static_cast<int64_t>(D.root_tok.size());
    const int64_t root_round = (L.stage_bytes - 64) / 8;
    for (int64_t i0 = 0; i0 < n_root; i0 += root_round) {
        const int64_t n = std::min(root_round, n_root - i0);
        const int64_t t_bytes = (n * 4 + 31) & ~int64_t(31);
        buf.resize(static_cast<size_t>(t_bytes + n * 4));
        std::memcpy(buf.data(), D.root_tok.data() + i0, static_cast<size_t>(n) * 4);
        std::memcpy(buf.data() + t_bytes, D.root_dst.data() + i0, static_cast<size_t>(n) * 4);
        SAM_CUDA(cudaMemcpyAsync(stage, buf.data(), buf.size(), cudaMemcpyHostToDevice, st));
        scatter_root_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(
            root, reinterpret_cast<const int32_t*>(stage), reinterpret_cast<const int32_t*>(stage + t_bytes),
            static_cast<int>(n), static_cast<int>(L.root_span));
        SAM_CUDA(cudaGetLastError());
        ++g_launches;
    }
    if (!D.corpus_tail.empty())
        SAM_CUDA(cudaMemcpyAsync(base + L.corpus_off + D.corpus_off * 4, D.corpus_tail.data(), D.corpus_tail.size() * 4,
                                 cudaMemcpyHostToDevice, st));
    return SAM_OK;
}

int apply_delta(sam_index* idx, const Delta& D, cudaStream_t st, const Renorm* rn = nullptr, bool* renormalized = nullptr) {
    if (D.status != SAM_OK) return D.status;
    bool did = false;
    const int rc = D.full ? apply_full(idx, D, st) : apply_changes(idx, D, st, rn, &did);
    if (renormalized) *renormalized = did;
    if (rc != SAM_OK) return rc;
    idx->dev.n_states = static_cast<int32_t>(D.n_states_after);
    idx->dev.n_corpus = D.n_tokens_after;
    idx->layout.n_states = D.n_states_after;
    idx->layout.n_corpus = D.n_tokens_after;
    return SAM_OK;
}

int upload_growing(sam_index* idx, void* device_buf, cudaStream_t st) {
    if (idx->ring) {       // nothing more is sent towards the blob that is being replaced
        std::lock_guard<std::mutex> lock(idx->ring->mu);
        idx->ring->enabled = false;
    }
    Delta image;
    int rc = dyn_full_image(idx, &image);
    if (rc != SAM_OK) return rc;
    idx->device_buf = device_buf;
    set_device_view(idx, device_buf);
    rc = apply_delta(idx, image, st);
    if (rc != SAM_OK) {
        idx->device_buf = nullptr;
        return rc;
    }
    char* base = static_cast<char*>(device_buf);
    SAM_CUDA(cudaMemsetAsync(base + idx->layout.ctrl_off, 0, 256, st));
    SAM_CUDA(cudaStreamSynchronize(st));
    return ring_attach(idx, base + idx->layout.ring_off);
}

// sam_sync with or without the repair of stream states at the end of the last update's kernel.
int sync_updates(sam_index* idx, cudaStream_t st, const Renorm* rn, int64_t* tokens_on_device) {
    std::vector<Delta> ready;
    {
        Delta D;
        while (dyn_pop_ready(idx, &D)) ready.push_back(std::move(D));
    }
    bool repaired = ready.empty();         // nothing changed: nothing to repair
    for (size_t i = 0; i < ready.size(); ++i) {
        const Delta& D = ready[i];
        const bool last = i + 1 == ready.size();
        bool did = false;
        const int rc = apply_delta(idx, D, st, last ? rn : nullptr, &did);
        if (rc != SAM_OK) return rc;
        if (last) repaired = did;
        if (D.full) {
            ++idx->updates_full;
            idx->update_bytes += static_cast<int64_t>(D.all_rec.size() * sizeof(StateRec) + D.all_wide.size() * sizeof(Edge) +
                                                      (D.all_root.size() + D.all_corpus.size()) * 4);
        } else {
            ++idx->updates_incremental;
            idx->update_bytes += static_cast<int64_t>(D.rec_ids.size() * 36 + D.seg_edges.size() * sizeof(Edge) +
                                                      D.segs.size() * sizeof(SegDesc) + D.root_tok.size() * 8 +
                                                      D.corpus_tail.size() * 4);
        }
    }
    if (rn && rn->B > 0 && !repaired) {
        // the last update went section by section (or was a whole image): the states are repaired by a kernel of their own
        renormalize_kernel<<<static_cast<unsigned>((rn->B + 127) / 128), 128, 0, st>>>(idx->dev, rn->B, rn->state, rn->matched_len);
        SAM_CUDA(cudaGetLastError());
        ++g_launches;
    }
    if (tokens_on_device) *tokens_on_device = idx->dev.n_corpus;
    return SAM_OK;
}

}  // namespace

struct sam_set {
    std::vector<const sam_index*> members;
    void* device_buf = nullptr;      // caller-owned table of DeviceSam
};

extern "C" {

int sam_build(const int32_t* corpus, int64_t n, const int32_t* separators, int32_t n_sep, sam_index** out) {
    if (!corpus || !out || n < 1 || n > (int64_t(1) << 29)) return SAM_ERR_INVALID_ARG;
    if (n_sep < 0 || n_sep > SAM_MAX_SEPARATORS || (n_sep > 0 && !separators)) return SAM_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i)
        if (corpus[i] < 0 || corpus[i] >= (1 << 24)) return SAM_ERR_INVALID_ARG;
    sam_index* idx = new (std::nothrow) sam_index();
    if (!idx) return SAM_ERR_NOMEM;
    const int rc = build_index(corpus, n, separators, n_sep, idx);
    if (rc != SAM_OK) {
        delete idx;
        return rc;
    }
    *out = idx;
    return SAM_OK;
}

int sam_sizes(const sam_index* idx, int64_t* n_states, int64_t* n_edges, int64_t* device_bytes) {
    if (!idx) return SAM_ERR_INVALID_ARG;
    if (idx->dyn) {
        const int rc = dyn_sizes(const_cast<sam_index*>(idx), n_states, n_edges);
        if (device_bytes) *device_bytes = idx->layout.total;
        return rc;
    }
    if (n_states) *n_states = idx->layout.n_states;
    if (n_edges) *n_edges = static_cast<int64_t>(idx->edge_tok.size());
    if (device_bytes) *device_bytes = idx->layout.total;
    return SAM_OK;
}

int sam_export(const sam_index* idx, int32_t* len, int32_t* link, int32_t* firstpos,
               int64_t* row_ptr, int32_t* edge_tok, int32_t* edge_dst) {
    if (!idx) return SAM_ERR_INVALID_ARG;
    if (idx->dyn) {
        const int rc = dyn_refresh_csr(const_cast<sam_index*>(idx));
        if (rc != SAM_OK) return rc;
    }
    const size_t S = idx->len.size(), E = idx->edge_tok.size();
    if (len) std::memcpy(len, idx->len.data(), S * 4);
    if (link) std::memcpy(link, idx->link.data(), S * 4);
    if (firstpos) std::memcpy(firstpos, idx->firstpos.data(), S * 4);
    if (row_ptr) std::memcpy(row_ptr, idx->row_ptr.data(), (S + 1) * 8);
    if (edge_tok) std::memcpy(edge_tok, idx->edge_tok.data(), E * 4);
    if (edge_dst) std::memcpy(edge_dst, idx->edge_dst.data(), E * 4);
    return SAM_OK;
}

int sam_upload(sam_index* idx, void* device_buf, int64_t bytes, void* cuda_stream) {
    if (!idx || !device_buf || !aligned(device_buf, 256)) return SAM_ERR_INVALID_ARG;
    const DeviceLayout& L = idx->layout;
    if (bytes < L.total) return SAM_ERR_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (idx->dyn) return upload_growing(idx, device_buf, st);
    std::vector<StateRec> rec;
    std::vector<Edge> wide;
    std::vector<int32_t> root;
    try {
        rec.resize(static_cast<size_t>(L.n_states));
        wide.resize(static_cast<size_t>(L.n_wide_edges));
        root.resize(static_cast<size_t>(L.root_span));
    } catch (const std::bad_alloc&) {
        return SAM_ERR_NOMEM;
    }
    pack_records(*idx, rec.data(), wide.data(), root.data());
    char* base = static_cast<char*>(device_buf);
    SAM_CUDA(cudaMemcpyAsync(base + L.rec_off, rec.data(), rec.size() * sizeof(StateRec), cudaMemcpyHostToDevice, st));
    if (!wide.empty())
        SAM_CUDA(cudaMemcpyAsync(base + L.edge_off, wide.data(), wide.size() * sizeof(Edge), cudaMemcpyHostToDevice, st));
    if (!root.empty())
        SAM_CUDA(cudaMemcpyAsync(base + L.root_off, root.data(), root.size() * 4, cudaMemcpyHostToDevice, st));
    SAM_CUDA(cudaMemcpyAsync(base + L.corpus_off, idx->corpus.data(), idx->corpus.size() * 4, cudaMemcpyHostToDevice, st));
    SAM_CUDA(cudaStreamSynchronize(st));
    idx->device_buf = device_buf;
    DeviceSam& d = idx->dev;
    d.rec = reinterpret_cast<const StateRec*>(base + L.rec_off);
    d.wide = reinterpret_cast<const Edge*>(base + L.edge_off);
    d.root_dst = reinterpret_cast<const int32_t*>(base + L.root_off);
    d.corpus = reinterpret_cast<const int32_t*>(base + L.corpus_off);
    d.root_span = static_cast<int32_t>(L.root_span);
    d.n_states = static_cast<int32_t>(L.n_states);
    d.n_corpus = L.n_corpus;
    d.n_sep = static_cast<int32_t>(idx->seps.size());
    for (int k = 0; k < SAM_MAX_SEPARATORS; ++k) d.seps[k] = (k < d.n_sep) ? idx->seps[k] : -1;
    return SAM_OK;
}

void sam_free(sam_index* idx) {
    if (!idx) return;
    if (idx->stage_event) {
        cudaEventSynchronize(static_cast<cudaEvent_t>(idx->stage_event));
        cudaEventDestroy(static_cast<cudaEvent_t>(idx->stage_event));
    }
    if (idx->pinned_stage) cudaFreeHost(idx->pinned_stage);
    dyn_destroy(idx);          // joins the builder thread, which may be sending an update to the ring
    ring_destroy(idx);
    delete idx;
}

int64_t sam_workspace_bytes(int32_t B, int32_t K) {
    if (B < 0 || K < 1 || K > SAM_K_MAX) return SAM_ERR_INVALID_ARG;
    return scratch_layout(nullptr, B, K).bytes;
}

int sam_workspace_init(void* workspace, int64_t bytes, void* cuda_stream) {
    if (!workspace || bytes < 0 || !aligned(workspace, 8)) return SAM_ERR_INVALID_ARG;
    SAM_CUDA(cudaMemsetAsync(workspace, 0, static_cast<size_t>(bytes), static_cast<cudaStream_t>(cuda_stream)));
    return SAM_OK;
}

int sam_draft(const sam_index* idx, int32_t B, int32_t* state, int32_t* matched_len,
              const int32_t* new_tokens, int32_t ld, const int32_t* n_new,
              int32_t K, int32_t min_match, int32_t* drafts, int32_t* n_draft, void* cuda_stream) {
    if (!idx || B < 0 || K < 1 || K > SAM_K_MAX || min_match < 1 || ld < 0) return SAM_ERR_INVALID_ARG;
    if (!idx->device_buf) return SAM_ERR_NOT_UPLOADED;
    if (B == 0) return SAM_OK;
    if (!state || !matched_len || !n_new || !drafts || !n_draft || (ld > 0 && !new_tokens)) return SAM_ERR_INVALID_ARG;
    const int warps = 4;
    const unsigned grid = static_cast<unsigned>((B + warps - 1) / warps);
    draft_kernel<<<grid, warps * 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        idx->dev, B, state, matched_len, new_tokens, ld, n_new, K, min_match, drafts, n_draft);
    ++g_launches;
    SAM_CUDA(cudaGetLastError());
    return SAM_OK;
}

int sam_verify_ex(const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                  const int32_t* drafts, const int32_t* n_draft,
                  int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                  uint32_t flags, int64_t* counters,
                  void* workspace, int64_t workspace_bytes, void* cuda_stream) {
    if (flags & ~static_cast<uint32_t>(SAM_STEP_NO_SPECULATION | SAM_STEP_SKIP_UNUSED_ROWS)) return SAM_ERR_INVALID_ARG;
    if (counters && !aligned(counters, 8)) return SAM_ERR_INVALID_ARG;
    int rc = check_verify_args(logits_bf16, row_stride_elems, B, K, V, drafts, n_draft, argmax_out, accepted,
                               n_accepted, workspace, workspace_bytes);
    if (rc != SAM_OK || B == 0) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int64_t R = static_cast<int64_t>(B) * (K + 1);
    const Scratch sc = scratch_layout(workspace, B, K);
    const AcceptArgs aa{static_cast<const __nv_bfloat16*>(logits_bf16), row_stride_elems, B, K, drafts, n_draft,
                        argmax_out, accepted, n_accepted, sc.keys, nullptr, nullptr, 1, nullptr, nullptr,
                        nullptr, nullptr, flags, reinterpret_cast<unsigned long long*>(counters)};
    RowMap rm{nullptr, nullptr, 0, 0, nullptr};
    if (flags & SAM_STEP_SKIP_UNUSED_ROWS) {
        build_row_list_kernel<<<1, 1024, 0, st>>>(n_draft, B, K, flags, sc.row_list, sc.list_meta);
        SAM_CUDA(cudaGetLastError());
        ++g_launches;
        rm = RowMap{sc.row_list, sc.list_meta, 0, row_list_sig(B, K), sc.status};
    }
    bool did_tail = false;
    rc = launch_argmax(logits_bf16, row_stride_elems, R, V, sc.keys, sc.status, st, nullptr, nullptr, nullptr,
                       &aa, kTailVerifyOnly, sc.done, &did_tail, &rm, sc.rowcnt, sc.acc_epoch, sc.list_meta + 8);
    if (rc != SAM_OK) return rc;
    if (!did_tail) {
        rc = launch_accept<kTailVerifyOnly>(DeviceSam{}, aa, st);
        if (rc != SAM_OK) return rc;
    }
    prof_mark(2, st);
    prof_done();
    return SAM_OK;
}

int sam_verify(const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
               const int32_t* drafts, const int32_t* n_draft,
               int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
               void* workspace, int64_t workspace_bytes, void* cuda_stream) {
    return sam_verify_ex(logits_bf16, row_stride_elems, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
                         0, nullptr, workspace, workspace_bytes, cuda_stream);
}

int sam_step_ex(const sam_index* idx,
                const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                const int32_t* drafts, const int32_t* n_draft,
                int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                int32_t* state, int32_t* matched_len, int32_t min_match,
                int32_t* next_drafts, int32_t* next_n_draft,
                uint32_t flags, int64_t* counters,
                void* workspace, int64_t workspace_bytes, void* cuda_stream) {
    if (!idx || min_match < 1) return SAM_ERR_INVALID_ARG;
    if (flags & ~static_cast<uint32_t>(SAM_STEP_NO_SPECULATION | SAM_STEP_SKIP_UNUSED_ROWS | SAM_STEP_ROW_LIST_READY))
        return SAM_ERR_INVALID_ARG;
    if ((flags & SAM_STEP_ROW_LIST_READY) && !(flags & SAM_STEP_SKIP_UNUSED_ROWS)) return SAM_ERR_INVALID_ARG;
    if (counters && !aligned(counters, 8)) return SAM_ERR_INVALID_ARG;
    int rc = check_verify_args(logits_bf16, row_stride_elems, B, K, V, drafts, n_draft, argmax_out, accepted,
                               n_accepted, workspace, workspace_bytes);
    if (rc != SAM_OK) return rc;
    if (!idx->device_buf) return SAM_ERR_NOT_UPLOADED;
    if (B == 0) return SAM_OK;
    if (!state || !matched_len || !next_drafts || !next_n_draft) return SAM_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int64_t R = static_cast<int64_t>(B) * (K + 1);
    const Scratch sc = scratch_layout(workspace, B, K);
    PreWalk pw{state, matched_len, drafts, n_draft, sc.pre_state, sc.pre_len, B, K, 1,
               (flags & SAM_STEP_NO_SPECULATION) ? 1 : 0};
    AcceptArgs aa{static_cast<const __nv_bfloat16*>(logits_bf16), row_stride_elems, B, K, drafts, n_draft,
                  argmax_out, accepted, n_accepted, sc.keys, state, matched_len, min_match, next_drafts,
                  next_n_draft, sc.pre_state, sc.pre_len, flags & (SAM_STEP_NO_SPECULATION | SAM_STEP_SKIP_UNUSED_ROWS),
                  reinterpret_cast<unsigned long long*>(counters), nullptr, nullptr};
    RowMap rm{nullptr, nullptr, 0, 0, nullptr};
    if (flags & SAM_STEP_SKIP_UNUSED_ROWS) {
        // the rows this step reads: listed by the previous step's accept kernel when the caller says so, else by a
        // small kernel in front; either way this step's accept kernel lists the rows of the next step
        // (with speculation off for this call the rows wanted are fewer than the previous step listed: list them afresh)
        if (!(flags & SAM_STEP_ROW_LIST_READY) || (flags & SAM_STEP_NO_SPECULATION)) {
            build_row_list_kernel<<<1, 1024, 0, st>>>(n_draft, B, K, flags, sc.row_list, sc.list_meta);
            SAM_CUDA(cudaGetLastError());
            ++g_launches;
        }
        rm = RowMap{sc.row_list, sc.list_meta, 0, row_list_sig(B, K), sc.status};
        aa.next_list = sc.row_list;
        aa.list_meta = sc.list_meta;
    }
    bool did_prewalk = false, did_tail = false;
    rc = launch_argmax(logits_bf16, row_stride_elems, R, V, sc.keys, sc.status, st, &idx->dev, &pw, &did_prewalk,
                       &aa, kTailResume, sc.done, &did_tail, &rm, sc.rowcnt, sc.acc_epoch, sc.list_meta + 8);
    if (rc != SAM_OK) return rc;
    if (!did_tail) {
        rc = did_prewalk ? launch_accept<kTailResume>(idx->dev, aa, st) : launch_accept<kTailFullWalk>(idx->dev, aa, st);
        if (rc != SAM_OK) return rc;
    }
    prof_mark(2, st);
    prof_done();
    return SAM_OK;
}

int sam_step(const sam_index* idx,
             const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
             const int32_t* drafts, const int32_t* n_draft,
             int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
             int32_t* state, int32_t* matched_len, int32_t min_match,
             int32_t* next_drafts, int32_t* next_n_draft,
             void* workspace, int64_t workspace_bytes, void* cuda_stream) {
    return sam_step_ex(idx, logits_bf16, row_stride_elems, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
                       state, matched_len, min_match, next_drafts, next_n_draft, 0, nullptr,
                       workspace, workspace_bytes, cuda_stream);
}

int sam_argmax_partial(const void* logits_bf16, int64_t row_stride_elems, int64_t rows, int32_t V, int32_t v_offset,
                       int64_t* keys, void* cuda_stream) {
    if (rows < 0 || V < 1 || row_stride_elems < V || v_offset < 0 || static_cast<int64_t>(v_offset) + V > (int64_t(1) << 31) - 1)
        return SAM_ERR_INVALID_ARG;
    if (rows == 0) return SAM_OK;
    if (!logits_bf16 || !keys || !aligned(logits_bf16, 2) || !aligned(keys, 8)) return SAM_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SAM_CUDA(cudaMemsetAsync(keys, 0, static_cast<size_t>(rows + 1) * 8, st));     // the last word is the status word
    const RowMap rm{nullptr, nullptr, v_offset, 0, nullptr};
    return launch_argmax(logits_bf16, row_stride_elems, rows, V, reinterpret_cast<unsigned long long*>(keys),
                         reinterpret_cast<int*>(keys + rows), st, nullptr, nullptr, nullptr, nullptr, 0, nullptr, nullptr, &rm);
}

int sam_step_from_keys(const sam_index* idx, int64_t* keys, int32_t B, int32_t K,
                       const int32_t* drafts, const int32_t* n_draft,
                       int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                       int32_t* state, int32_t* matched_len, int32_t min_match,
                       int32_t* next_drafts, int32_t* next_n_draft, void* cuda_stream) {
    if (!idx || B < 0 || K < 1 || K > SAM_K_MAX || min_match < 1) return SAM_ERR_INVALID_ARG;
    if (!idx->device_buf) return SAM_ERR_NOT_UPLOADED;
    if (B == 0) return SAM_OK;
    if (!keys || !aligned(keys, 8) || !drafts || !n_draft || !argmax_out || !accepted || !n_accepted || !state ||
        !matched_len || !next_drafts || !next_n_draft)
        return SAM_ERR_INVALID_ARG;
    const AcceptArgs aa{nullptr, 0, B, K, drafts, n_draft, argmax_out, accepted, n_accepted,
                        reinterpret_cast<unsigned long long*>(keys), state, matched_len, min_match, next_drafts,
                        next_n_draft, nullptr, nullptr, 0u, nullptr};
    return launch_accept<kTailFullWalk>(idx->dev, aa, static_cast<cudaStream_t>(cuda_stream), false);
}

int64_t sam_set_bytes(int32_t n_members) {
    if (n_members < 1) return SAM_ERR_INVALID_ARG;
    return (static_cast<int64_t>(n_members) * static_cast<int64_t>(sizeof(DeviceSam)) + 255) & ~int64_t(255);
}

int sam_set_refresh(sam_set* set, void* cuda_stream) {
    if (!set || !set->device_buf) return SAM_ERR_INVALID_ARG;
    std::vector<DeviceSam> table(set->members.size());
    for (size_t i = 0; i < set->members.size(); ++i) {
        if (!set->members[i]->device_buf) return SAM_ERR_NOT_UPLOADED;
        table[i] = set->members[i]->dev;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SAM_CUDA(cudaMemcpyAsync(set->device_buf, table.data(), table.size() * sizeof(DeviceSam), cudaMemcpyHostToDevice, st));
    return SAM_OK;
}

int sam_set_create(const sam_index* const* members, int32_t n_members, void* device_buf, int64_t bytes,
                   void* cuda_stream, sam_set** out) {
    if (!members || n_members < 1 || !device_buf || !out || !aligned(device_buf, 16)) return SAM_ERR_INVALID_ARG;
    if (bytes < sam_set_bytes(n_members)) return SAM_ERR_TOO_SMALL;
    for (int32_t i = 0; i < n_members; ++i)
        if (!members[i]) return SAM_ERR_INVALID_ARG;
    sam_set* set = new (std::nothrow) sam_set();
    if (!set) return SAM_ERR_NOMEM;
    set->members.assign(members, members + n_members);
    set->device_buf = device_buf;
    const int rc = sam_set_refresh(set, cuda_stream);
    if (rc != SAM_OK) {
        delete set;
        return rc;
    }
    *out = set;
    return SAM_OK;
}

void sam_set_free(sam_set* set) { delete set; }

int sam_set_renormalize(const sam_set* set, int32_t member, int32_t B, int32_t M, const int32_t* slots,
                        int32_t* state, const int32_t* matched_len, void* cuda_stream) {
    if (!set || member < 0 || member >= static_cast<int32_t>(set->members.size()) || B < 0 || M < 1 || M > kMaxSlots)
        return SAM_ERR_INVALID_ARG;
    const sam_index* idx = set->members[member];
    if (!idx->device_buf) return SAM_ERR_NOT_UPLOADED;
    if (B == 0) return SAM_OK;
    if (!slots || !state || !matched_len) return SAM_ERR_INVALID_ARG;
    const int n = B * M;
    renormalize_slots_kernel<<<static_cast<unsigned>((n + 127) / 128), 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        idx->dev, member, n, slots, state, matched_len);
    SAM_CUDA(cudaGetLastError());
    ++g_launches;
    return SAM_OK;
}

int sam_multi_draft(const sam_set* set, int32_t B, int32_t M, const int32_t* slots, const float* weights,
                    int32_t* state, int32_t* matched_len, const int32_t* new_tokens, int32_t ld, const int32_t* n_new,
                    int32_t K, int32_t min_match, int32_t* drafts, int32_t* n_draft, int32_t* chosen,
                    void* cuda_stream) {
    if (!set || B < 0 || M < 1 || M > kMaxSlots || K < 1 || K > SAM_K_MAX || min_match < 1 || ld < 0)
        return SAM_ERR_INVALID_ARG;
    if (B == 0) return SAM_OK;
    if (!slots || !weights || !state || !matched_len || !n_new || !drafts || !n_draft || !chosen || (ld > 0 && !new_tokens))
        return SAM_ERR_INVALID_ARG;
    multi_draft_kernel<<<static_cast<unsigned>(B), 32 * M, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const DeviceSam*>(set->device_buf), static_cast<int>(set->members.size()), B, M, slots, weights,
        state, matched_len, new_tokens, ld, n_new, K, min_match, drafts, n_draft, chosen);
    SAM_CUDA(cudaGetLastError());
    ++g_launches;
    return SAM_OK;
}

int64_t sam_multi_workspace_bytes(int32_t B, int32_t K, int32_t M) {
    if (B < 0 || K < 1 || K > SAM_K_MAX || M < 1 || M > kMaxSlots) return SAM_ERR_INVALID_ARG;
    return scratch_layout(nullptr, B, K, M).bytes;
}

int sam_multi_step(const sam_set* set,
                   const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                   const int32_t* drafts, const int32_t* n_draft,
                   int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                   int32_t M, const int32_t* slots, const float* weights, int32_t* state, int32_t* matched_len,
                   int32_t min_match, int32_t* next_drafts, int32_t* next_n_draft, int32_t* chosen,
                   void* workspace, int64_t workspace_bytes, void* cuda_stream) {
    if (!set || M < 1 || M > kMaxSlots || min_match < 1) return SAM_ERR_INVALID_ARG;
    if (B < 0 || K < 1 || K > SAM_K_MAX || V < 1 || row_stride_elems < V) return SAM_ERR_INVALID_ARG;
    if (B == 0) return SAM_OK;
    if (!logits_bf16 || !drafts || !n_draft || !argmax_out || !accepted || !n_accepted || !slots || !weights || !state ||
        !matched_len || !next_drafts || !next_n_draft || !chosen || !workspace || !aligned(logits_bf16, 2) ||
        !aligned(workspace, 8))
        return SAM_ERR_INVALID_ARG;
    if (workspace_bytes < sam_multi_workspace_bytes(B, K, M)) return SAM_ERR_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int64_t R = static_cast<int64_t>(B) * (K + 1);
    const Scratch sc = scratch_layout(workspace, B, K, M);
    const DeviceSam* table = static_cast<const DeviceSam*>(set->device_buf);
    const int n_members = static_cast<int>(set->members.size());
    PreWalk pw{state, matched_len, drafts, n_draft, sc.pre_state, sc.pre_len, B, K, 1, 0, table, slots, M, n_members};
    bool did_prewalk = false;
    int rc = launch_argmax(logits_bf16, row_stride_elems, R, V, sc.keys, sc.status, st, nullptr, &pw, &did_prewalk);
    if (rc != SAM_OK) return rc;
    if (!did_prewalk) {
        // the direct-load argmax kernel has no spare warps: the slots walk the whole accepted run afterwards
        const AcceptArgs aa{static_cast<const __nv_bfloat16*>(logits_bf16), row_stride_elems, B, K, drafts, n_draft,
                            argmax_out, accepted, n_accepted, sc.keys, nullptr, nullptr, 1, nullptr, nullptr,
                            nullptr, nullptr, 0u, nullptr};
        rc = launch_accept<kTailVerifyOnly>(DeviceSam{}, aa, st);
        if (rc != SAM_OK) return rc;
        multi_draft_kernel<<<static_cast<unsigned>(B), 32 * M, 0, st>>>(
            table, n_members, B, M, slots, weights, state, matched_len, accepted, K + 1, n_accepted, K, min_match,
            next_drafts, next_n_draft, chosen);
        SAM_CUDA(cudaGetLastError());
        ++g_launches;
    } else {
        const AcceptArgs aa{static_cast<const __nv_bfloat16*>(logits_bf16), row_stride_elems, B, K, drafts, n_draft,
                            argmax_out, accepted, n_accepted, sc.keys, nullptr, nullptr, min_match, next_drafts,
                            next_n_draft, nullptr, nullptr, 0u, nullptr};
        const MultiArgs ma{table, n_members, M, slots, weights, state, matched_len, sc.pre_state, sc.pre_len, chosen};
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(B));
        cfg.blockDim = dim3(32 * M);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        SAM_CUDA(cudaLaunchKernelEx(&cfg, multi_step_kernel, aa, ma));
        ++g_launches;
    }
    prof_mark(2, st);
    prof_done();
    return SAM_OK;
}

int sam_adaptive_switch(int64_t context_len, int64_t batch_size, int64_t max_context_len, int64_t max_batch_size) {
    return (context_len > max_context_len || batch_size > max_batch_size) ? 0 : 1;
}

int sam_speculation_pays(const int64_t* counters, int32_t K, double cost_ratio) {
    if (!counters || K < 1 || K > SAM_K_MAX || !(cost_ratio > 0.0)) return SAM_ERR_INVALID_ARG;
    const int64_t passes = counters[0], accepted_drafts = counters[3], rows_read = counters[5];
    if (passes < 0 || accepted_drafts < 0 || rows_read < passes) return SAM_ERR_INVALID_ARG;
    if (passes == 0) return 1;                       // an empty window is no evidence against speculating
    // tokens gained over plain decoding, scaled by K, against the extra rows read, priced at (cost_ratio - 1) / K each
    const double gain = static_cast<double>(accepted_drafts) * static_cast<double>(K);
    const double extra_cost = (cost_ratio - 1.0) * static_cast<double>(rows_read - passes);
    return gain > extra_cost ? 1 : 0;
}

namespace {
struct HostStepLayout {
    int64_t logits, drafts, n_draft, argmax, accepted, n_accepted, state, mlen, ws, total;
    int64_t logits_bytes, ws_bytes;
};
bool host_step_layout(int64_t stride, int32_t B, int32_t K, int32_t V, HostStepLayout* L) {
    if (B < 0 || K < 1 || K > SAM_K_MAX || V < 1 || stride < V) return false;
    auto up = [](int64_t x) { return (x + 255) & ~int64_t(255); };
    const int64_t R = static_cast<int64_t>(B) * (K + 1);
    L->logits_bytes = R > 0 ? ((R - 1) * stride + V) * 2 : 0;
    L->ws_bytes = sam_workspace_bytes(B, K);
    int64_t o = 0;
    L->logits = o;     o = up(o + L->logits_bytes + 16);
    L->drafts = o;     o = up(o + static_cast<int64_t>(B) * K * 4);
    L->n_draft = o;    o = up(o + static_cast<int64_t>(B) * 4);
    L->argmax = o;     o = up(o + R * 4);
    L->accepted = o;   o = up(o + R * 4);
    L->n_accepted = o; o = up(o + static_cast<int64_t>(B) * 4);
    L->state = o;      o = up(o + static_cast<int64_t>(B) * 4);
    L->mlen = o;       o = up(o + static_cast<int64_t>(B) * 4);
    L->ws = o;         o = up(o + L->ws_bytes);
    L->total = o;
    return true;
}
}  // namespace

// ---- allocation-free verification ------------------------------------------------------------
// The scratch words live in the library image: one array per GPU that loads the module, zero at
// load time, shared by every sam_verify_static call on that GPU.
static __device__ __align__(256) unsigned long long g_static_keys[SAM_STATIC_MAX_ROWS + 32];   // + status word

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
unsigned long long* g_static_keys_addr[kMaxDevices] = {};   // device address of g_static_keys, per device

// In host code `g_static_keys` is only a handle for the runtime, not an address a kernel can use:
// the real device address is looked up once per device, with that device current.
int static_scratch(unsigned long long** out) {
    int dev = -1;
    SAM_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SAM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_keys_addr[dev]) {
        unsigned long long* ptr = nullptr;
        SAM_CUDA(cudaGetSymbolAddress((void**)&ptr, g_static_keys));
        g_static_keys_addr[dev] = ptr;
    }
    *out = g_static_keys_addr[dev];
    return SAM_OK;
}
}  // namespace

int sam_verify_static(const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                      const int32_t* drafts, const int32_t* n_draft,
                      int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted, void* cuda_stream) {
    if (B < 0 || K < 1 || K > SAM_K_MAX) return SAM_ERR_INVALID_ARG;
    const int64_t rows = static_cast<int64_t>(B) * (K + 1);
    if (rows > SAM_STATIC_MAX_ROWS) return SAM_ERR_TOO_LARGE;
    unsigned long long* keys = nullptr;
    int rc = static_scratch(&keys);
    if (rc != SAM_OK) return rc;
    rc = check_verify_args(logits_bf16, row_stride_elems, B, K, V, drafts, n_draft, argmax_out, accepted,
                           n_accepted, keys, INT64_MAX);   // the array is sized for SAM_STATIC_MAX_ROWS rows
    if (rc != SAM_OK || B == 0) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // whatever an earlier (possibly failed) call left behind, these rows and the status word start from zero
    SAM_CUDA(cudaMemsetAsync(keys, 0, static_cast<size_t>(rows) * 8, st));
    SAM_CUDA(cudaMemsetAsync(keys + SAM_STATIC_MAX_ROWS, 0, sizeof(int), st));
    rc = launch_argmax(logits_bf16, row_stride_elems, rows, V, keys,
                       reinterpret_cast<int*>(keys + SAM_STATIC_MAX_ROWS), st);
    if (rc != SAM_OK) return rc;
    const AcceptArgs aa{static_cast<const __nv_bfloat16*>(logits_bf16), row_stride_elems, B, K, drafts, n_draft,
                        argmax_out, accepted, n_accepted, keys, nullptr, nullptr, 1, nullptr, nullptr,
                        nullptr, nullptr, 0u, nullptr};
    rc = launch_accept<kTailVerifyOnly>(DeviceSam{}, aa, st);
    if (rc != SAM_OK) return rc;
    prof_mark(2, st);
    prof_done();
    return SAM_OK;
}

int sam_static_status(int32_t* status_out, void* cuda_stream) {
    if (!status_out) return SAM_ERR_INVALID_ARG;
    unsigned long long* keys = nullptr;
    const int rc = static_scratch(&keys);
    if (rc != SAM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SAM_CUDA(cudaMemcpyAsync(status_out, keys + SAM_STATIC_MAX_ROWS, sizeof(int), cudaMemcpyDeviceToHost, st));
    SAM_CUDA(cudaStreamSynchronize(st));
    return SAM_OK;
}

int64_t sam_step_host_staging_bytes(int64_t row_stride_elems, int32_t B, int32_t K, int32_t V) {
    HostStepLayout L;
    if (!host_step_layout(row_stride_elems, B, K, V, &L)) return SAM_ERR_INVALID_ARG;
    return L.total;
}

int sam_step_host(const sam_index* idx,
                  const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                  const int32_t* drafts, const int32_t* n_draft,
                  int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                  int32_t* state, int32_t* matched_len, int32_t min_match,
                  int32_t* next_drafts, int32_t* next_n_draft,
                  void* staging, int64_t staging_bytes, void* cuda_stream) {
    return sam_step_host_ex(idx, logits_bf16, row_stride_elems, B, K, V, drafts, n_draft, argmax_out, accepted, n_accepted,
                            state, matched_len, min_match, next_drafts, next_n_draft, 0, staging, staging_bytes, cuda_stream);
}

int sam_step_host_ex(const sam_index* idx,
                     const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                     const int32_t* drafts, const int32_t* n_draft,
                     int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                     int32_t* state, int32_t* matched_len, int32_t min_match,
                     int32_t* next_drafts, int32_t* next_n_draft, uint32_t flags,
                     void* staging, int64_t staging_bytes, void* cuda_stream) {
    HostStepLayout L;
    if (flags & ~static_cast<uint32_t>(SAM_STEP_NO_SPECULATION | SAM_STEP_SKIP_UNUSED_ROWS)) return SAM_ERR_INVALID_ARG;
    if (!idx || !host_step_layout(row_stride_elems, B, K, V, &L) || min_match < 1) return SAM_ERR_INVALID_ARG;
    if (!idx->device_buf) return SAM_ERR_NOT_UPLOADED;
    if (B == 0) return SAM_OK;
    if (!logits_bf16 || !drafts || !n_draft || !argmax_out || !accepted || !n_accepted || !state || !matched_len ||
        !next_drafts || !next_n_draft || !staging || !aligned(staging, 256))
        return SAM_ERR_INVALID_ARG;
    if (staging_bytes < L.total) return SAM_ERR_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* d = static_cast<char*>(staging);
    const size_t bB = static_cast<size_t>(B) * 4, bK = bB * K, bR = bB * (K + 1);
    if (flags & SAM_STEP_SKIP_UNUSED_ROWS) {
        // only the rows the step will read cross the bus: rows 0..n_draft[b] of every stream.  Runs of rows that touch
        // (a full proposal is followed directly by the next stream's rows) or that are less than a row apart go in one
        // copy - a copy costs a few microseconds of its own, about what a row takes on the bus
        const char* src = static_cast<const char*>(logits_bf16);
        const int64_t row_bytes = row_stride_elems * 2;
        int64_t run_first = -1, run_end = 0;            // byte range [run_first, run_end) waiting to be copied
        for (int32_t b = 0; b < B; ++b) {
            int32_t nd = (flags & SAM_STEP_NO_SPECULATION) ? 0 : n_draft[b];
            nd = nd < 0 ? 0 : (nd > K ? K : nd);
            const int64_t first = static_cast<int64_t>(b) * (K + 1) * row_bytes;
            const int64_t end = first + static_cast<int64_t>(nd) * row_bytes + static_cast<int64_t>(V) * 2;
            if (run_first >= 0 && first - run_end <= row_bytes) {
                run_end = end;
                continue;
            }
            if (run_first >= 0)
                SAM_CUDA(cudaMemcpyAsync(d + L.logits + run_first, src + run_first, static_cast<size_t>(run_end - run_first),
                                         cudaMemcpyHostToDevice, st));
            run_first = first;
            run_end = end;
        }
        if (run_first >= 0)
            SAM_CUDA(cudaMemcpyAsync(d + L.logits + run_first, src + run_first, static_cast<size_t>(run_end - run_first),
                                     cudaMemcpyHostToDevice, st));
    } else {
        SAM_CUDA(cudaMemcpyAsync(d + L.logits, logits_bf16, static_cast<size_t>(L.logits_bytes), cudaMemcpyHostToDevice, st));
    }
    SAM_CUDA(cudaMemcpyAsync(d + L.drafts, drafts, bK, cudaMemcpyHostToDevice, st));
    SAM_CUDA(cudaMemcpyAsync(d + L.n_draft, n_draft, bB, cudaMemcpyHostToDevice, st));
    SAM_CUDA(cudaMemcpyAsync(d + L.state, state, bB, cudaMemcpyHostToDevice, st));
    SAM_CUDA(cudaMemcpyAsync(d + L.mlen, matched_len, bB, cudaMemcpyHostToDevice, st));
    SAM_CUDA(cudaMemsetAsync(d + L.ws, 0, static_cast<size_t>(L.ws_bytes), st));
    int32_t* dd = reinterpret_cast<int32_t*>(d + L.drafts);
    int32_t* dn = reinterpret_cast<int32_t*>(d + L.n_draft);
    const int rc = sam_step_ex(idx, d + L.logits, row_stride_elems, B, K, V, dd, dn,
                               reinterpret_cast<int32_t*>(d + L.argmax), reinterpret_cast<int32_t*>(d + L.accepted),
                               reinterpret_cast<int32_t*>(d + L.n_accepted), reinterpret_cast<int32_t*>(d + L.state),
                               reinterpret_cast<int32_t*>(d + L.mlen), min_match, dd, dn, flags, nullptr,
                               d + L.ws, L.ws_bytes, st);
    if (rc != SAM_OK) return rc;
    SAM_CUDA(cudaMemcpyAsync(argmax_out, d + L.argmax, bR, cudaMemcpyDeviceToHost, st));
    SAM_CUDA(cudaMemcpyAsync(accepted, d + L.accepted, bR, cudaMemcpyDeviceToHost, st));
    SAM_CUDA(cudaMemcpyAsync(n_accepted, d + L.n_accepted, bB, cudaMemcpyDeviceToHost, st));
    SAM_CUDA(cudaMemcpyAsync(state, d + L.state, bB, cudaMemcpyDeviceToHost, st));
    SAM_CUDA(cudaMemcpyAsync(matched_len, d + L.mlen, bB, cudaMemcpyDeviceToHost, st));
    SAM_CUDA(cudaMemcpyAsync(next_drafts, d + L.drafts, bK, cudaMemcpyDeviceToHost, st));
    SAM_CUDA(cudaMemcpyAsync(next_n_draft, d + L.n_draft, bB, cudaMemcpyDeviceToHost, st));
    SAM_CUDA(cudaStreamSynchronize(st));
    return SAM_OK;
}

int sam_build_growing(const int32_t* corpus, int64_t n, const int32_t* separators, int32_t n_sep,
                      int64_t max_tokens, int32_t max_token_id, sam_index** out) {
    if (!out || n < 0 || (n > 0 && !corpus)) return SAM_ERR_INVALID_ARG;
    if (n_sep < 0 || n_sep > SAM_MAX_SEPARATORS || (n_sep > 0 && !separators)) return SAM_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i)
        if (corpus[i] < 0) return SAM_ERR_INVALID_ARG;
    sam_index* idx = new (std::nothrow) sam_index();
    if (!idx) return SAM_ERR_NOMEM;
    idx->seps.assign(separators, separators + n_sep);
    const int rc = dyn_create(idx, corpus, n, max_tokens, max_token_id);
    if (rc != SAM_OK) {
        delete idx;
        return rc;
    }
    *out = idx;
    return SAM_OK;
}

int sam_extend_async(sam_index* idx, const int32_t* tokens, int64_t n) {
    if (!idx || !idx->dyn) return SAM_ERR_INVALID_ARG;
    return dyn_enqueue(idx, tokens, n);
}

int sam_extend(sam_index* idx, const int32_t* tokens, int64_t n) {
    if (!idx || !idx->dyn) return SAM_ERR_INVALID_ARG;
    const int rc = dyn_enqueue(idx, tokens, n);
    if (rc != SAM_OK) return rc;
    return dyn_wait(idx);
}

int sam_pending(sam_index* idx, int64_t* tokens_queued, int64_t* tokens_built, int64_t* tokens_on_device) {
    if (!idx || !idx->dyn) return SAM_ERR_INVALID_ARG;
    dyn_counts(idx, tokens_queued, tokens_built);
    if (tokens_on_device) *tokens_on_device = idx->device_buf ? idx->dev.n_corpus : 0;
    return SAM_OK;
}

int sam_sync(sam_index* idx, void* cuda_stream, int64_t* tokens_on_device) {
    if (!idx || !idx->dyn) return SAM_ERR_INVALID_ARG;
    if (!idx->device_buf) return SAM_ERR_NOT_UPLOADED;
    return sync_updates(idx, static_cast<cudaStream_t>(cuda_stream), nullptr, tokens_on_device);
}

int sam_sync_renormalize(sam_index* idx, int32_t B, int32_t* state, const int32_t* matched_len, void* cuda_stream,
                         int64_t* tokens_on_device) {
    if (!idx || !idx->dyn || B < 0) return SAM_ERR_INVALID_ARG;
    if (!idx->device_buf) return SAM_ERR_NOT_UPLOADED;
    if (B > 0 && (!state || !matched_len)) return SAM_ERR_INVALID_ARG;
    const Renorm rn{B, state, matched_len};
    return sync_updates(idx, static_cast<cudaStream_t>(cuda_stream), &rn, tokens_on_device);
}

int sam_update_stats(const sam_index* idx, int64_t* incremental, int64_t* full_images, int64_t* bytes_copied) {
    if (!idx || !idx->dyn) return SAM_ERR_INVALID_ARG;
    if (incremental) *incremental = idx->updates_incremental;
    if (full_images) *full_images = idx->updates_full;
    if (bytes_copied) *bytes_copied = idx->update_bytes;
    return SAM_OK;
}

int sam_growing_set_relayout_every(sam_index* idx, int64_t every) {
    if (!idx || !idx->dyn) return SAM_ERR_INVALID_ARG;
    return dyn_set_relayout_every(idx, every);
}

int sam_renormalize(const sam_index* idx, int32_t B, int32_t* state, const int32_t* matched_len, void* cuda_stream) {
    if (!idx || B < 0) return SAM_ERR_INVALID_ARG;
    if (!idx->device_buf) return SAM_ERR_NOT_UPLOADED;
    if (B == 0) return SAM_OK;
    if (!state || !matched_len) return SAM_ERR_INVALID_ARG;
    renormalize_kernel<<<static_cast<unsigned>((B + 127) / 128), 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        idx->dev, B, state, matched_len);
    SAM_CUDA(cudaGetLastError());
    ++g_launches;
    return SAM_OK;
}

int sam_profile_enable(int32_t max_calls) {
    if (max_calls < 0) return SAM_ERR_INVALID_ARG;
    for (cudaEvent_t e : g_prof.ev) cudaEventDestroy(e);
    g_prof.ev.clear();
    g_prof.cap = g_prof.used = 0;
    try {
        g_prof.ev.reserve(static_cast<size_t>(max_calls) * 3);
    } catch (const std::bad_alloc&) {
        return SAM_ERR_NOMEM;
    }
    for (int64_t i = 0; i < static_cast<int64_t>(max_calls) * 3; ++i) {
        cudaEvent_t e;
        SAM_CUDA(cudaEventCreate(&e));
        g_prof.ev.push_back(e);
    }
    g_prof.cap = max_calls;
    return SAM_OK;
}

int32_t sam_profile_count(void) { return g_prof.used; }

int sam_profile_read(int32_t call, float* argmax_ms, float* accept_ms) {
    if (call < 0 || call >= g_prof.used) return SAM_ERR_INVALID_ARG;
    const size_t o = static_cast<size_t>(call) * 3;
    if (argmax_ms) SAM_CUDA(cudaEventElapsedTime(argmax_ms, g_prof.ev[o], g_prof.ev[o + 1]));
    if (accept_ms) SAM_CUDA(cudaEventElapsedTime(accept_ms, g_prof.ev[o + 1], g_prof.ev[o + 2]));
    return SAM_OK;
}

int sam_workspace_status(const void* workspace, int32_t B, int32_t K, int32_t* status_out, void* cuda_stream) {
    if (!workspace || !status_out || B < 0 || K < 1 || K > SAM_K_MAX) return SAM_ERR_INVALID_ARG;
    const int64_t R = static_cast<int64_t>(B) * (K + 1);
    const int* w = status_word(static_cast<unsigned long long*>(const_cast<void*>(workspace)), R);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SAM_CUDA(cudaMemcpyAsync(status_out, w, sizeof(int), cudaMemcpyDeviceToHost, st));
    SAM_CUDA(cudaStreamSynchronize(st));
    return SAM_OK;
}

int sam_set_argmax_variant(int32_t variant) {
    if (variant < 0 || variant > 3) return SAM_ERR_INVALID_ARG;
    g_argmax_variant = variant;
    return SAM_OK;
}

const char* sam_strerror(int status) {
    switch (status) {
        case SAM_OK: return "ok";
        case SAM_ERR_INVALID_ARG: return "invalid argument";
        case SAM_ERR_NOMEM: return "out of host memory";
        case SAM_ERR_NOT_UPLOADED: return "automaton not uploaded to the device";
        case SAM_ERR_CUDA: return "CUDA call failed";
        case SAM_ERR_TOO_SMALL: return "caller buffer too small";
        case SAM_ERR_TOO_LARGE: return "size exceeds a built-in limit of this entry point";
        default: return "unknown status";
    }
}

int sam_last_cuda_error(void) { return g_last_cuda; }

int64_t sam_launch_count(void) { return g_launches.load(); }

}  // extern "C"
