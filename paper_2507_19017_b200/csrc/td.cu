// Host side of the C ABI declared in include/td.h: argument checks, workspace carving and
// kernel launches.  No device memory is allocated here and nothing synchronises except
// td_create (once) and td_status.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "td_device.cuh"
#include "td_get.cuh"
#include "td_put.cuh"

using namespace td;

// Named ranges around the public calls for timeline tools (NVTX; compiled in with -DTD_NVTX, the
// header-only nvtx3 that ships with the toolkit; otherwise the macro is empty).
#ifdef TD_NVTX
#include <nvtx3/nvToolsExt.h>
namespace {
struct TdRange {
    explicit TdRange(const char *name) { nvtxRangePushA(name); }
    ~TdRange() { nvtxRangePop(); }
};
}  // namespace
#define TD_RANGE(name) TdRange td_range_guard(name)
#else
#define TD_RANGE(name) do { } while (0)
#endif

struct td_dock {
    DockView dv;
    td_config cfg;                 // columns / consumers pointers are not kept
    int device;
    int sm_count;
    uint8_t *ws;
    size_t ws_bytes;
    size_t table_bytes[7];
    std::atomic<uint64_t> launches;
    std::mutex slot_mu;
    std::vector<cudaStream_t> slot_stream;     // which stream draws from which scatter chunk counter
    std::mutex put_mu;                         // a put takes its number and enqueues its kernels as one step
    // optional per-kernel timing of the two copy kernels (0 = put scatter, 1 = get gather)
    std::atomic<bool> timing;
    std::mutex timing_mu;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> timing_ev[2];
};

namespace {

std::atomic<uint32_t> g_seq{1};     // launch sequence numbers for scan scratch, process wide
std::atomic<unsigned long long> g_put_seq{1};         // numbers of the puts that tell their scatter kernel when to look
constexpr uint32_t kDefaultPollLimit = 1u << 20;      // polls before a device-side wait gives up (tens of milliseconds)

inline size_t align_up_sz(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline uint32_t esize_of(int32_t dtype) { return dtype == TD_BF16 ? 2u : 4u; }

// Dynamic shared memory of the copy kernels: the warps' stages and mbarriers, then (gather) the
// block-scan scratch and the job table.
constexpr size_t kStageSmem = (size_t)kCopyWarps * kPipeSmemPerWarp;
size_t scatter_smem_bytes() { return kStageSmem; }
size_t gather_smem_bytes(uint32_t n_req, uint32_t jobs_per_req) {
    return kStageSmem + (size_t)kCopyWarps * 8 + (size_t)n_req * jobs_per_req * 4 + (size_t)n_req * 4;
}

struct Layout {
    size_t status, len[3], off[3], cursor[3], claim, consumed, errword, counters, put_counters, put_ready, progress,
           col[kMaxColumns], total;
    uint32_t claim_words, consumed_words;
    uint64_t cap[3];
};

bool valid_config(const td_config *c) {
    if (!c || !c->columns || !c->consumers) return false;
    if (c->n_prompts == 0 || c->n_per_group == 0 || c->n_shards == 0 || c->n_shards > 256) return false;
    if (c->n_prompts % c->n_shards) return false;
    if (c->n_columns == 0 || c->n_columns > 32 || c->n_consumers == 0 || c->n_consumers > 32) return false;
    if ((uint64_t)c->n_prompts * c->n_per_group >= (1ull << 30)) return false;
    for (uint32_t k = 0; k < c->n_columns; ++k) {
        const td_column &col = c->columns[k];
        if (col.dtype < TD_I32 || col.dtype > TD_BF16) return false;
        if (col.cls < TD_SCALAR || col.cls > TD_RESPONSE) return false;
    }
    const uint32_t all = c->n_columns == 32 ? 0xffffffffu : ((1u << c->n_columns) - 1u);
    for (uint32_t k = 0; k < c->n_consumers; ++k) {
        const td_consumer &q = c->consumers[k];
        if ((q.need_mask & ~all) || (q.out_mask & ~q.need_mask)) return false;
        if (q.flags & TD_F_ADVANTAGE) {
            if (c->reward_column >= c->n_columns) return false;
            const td_column &r = c->columns[c->reward_column];
            if (r.cls != TD_SCALAR || r.dtype != TD_F32) return false;
            if (!((q.need_mask >> c->reward_column) & 1u)) return false;
        }
    }
    return true;
}

Layout make_layout(const td_config *c) {
    Layout L{};
    const size_t n = (size_t)c->n_prompts * c->n_per_group;
    const size_t S = c->n_shards;
    L.cap[1] = (c->prompt_elems_per_shard + 7) / 8 * 8;
    L.cap[2] = (c->response_elems_per_shard + 7) / 8 * 8;
    L.claim_words = (c->n_prompts + 31) / 32;
    L.consumed_words = (uint32_t)((n + 31) / 32);
    size_t p = 0;
    auto take = [&](size_t bytes) { size_t at = p; p = align_up_sz(p + bytes, 256); return at; };
    L.errword = take(256);
    L.counters = take(CNT_TOTAL * 8);
    L.put_counters = take((size_t)kPutCounterSlots * 8);
    L.put_ready = take((size_t)kPutCounterSlots * 4 * 8);
    L.progress = take((size_t)c->n_columns * n * 4);
    L.status = take(n * 4);
    for (int k = 1; k <= 2; ++k) { L.len[k] = take(n * 4); L.off[k] = take(n * 8); L.cursor[k] = take(S * 8); }
    L.claim = take((size_t)c->n_consumers * L.claim_words * 4);
    L.consumed = take((size_t)c->n_consumers * L.consumed_words * 4);
    for (uint32_t k = 0; k < c->n_columns; ++k) {
        const td_column &col = c->columns[k];
        const size_t es = esize_of(col.dtype);
        L.col[k] = take(col.cls == TD_SCALAR ? n * es : S * L.cap[col.cls] * es);
    }
    L.total = p;
    return L;
}

template <typename... KArgs, typename... Args>
cudaError_t launch(td_dock *d, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                   cudaStream_t st, Args &&...args) {
    kernel<<<grid, block, smem, st>>>(std::forward<Args>(args)...);
    d->launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

// Launch of a kernel that may be brought on before the kernel ahead of it in the stream has
// finished (programmatic dependent launch); the kernel itself waits, with griddep_wait(), before
// it touches that kernel's results.
template <typename... KArgs, typename... Args>
cudaError_t launch_dep(td_dock *d, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t st, Args &&...args) {
#ifdef TD_NO_PDL
    return launch(d, kernel, grid, block, smem, st, std::forward<Args>(args)...);
#endif
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    d->launches.fetch_add(1, std::memory_order_relaxed);
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

// Launch bracketed by a pair of events on the same stream while timing is switched on.
template <typename... KArgs, typename... Args>
cudaError_t launch_timed(td_dock *d, int which, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                         cudaStream_t st, Args &&...args) {
    if (!d->timing.load(std::memory_order_relaxed))
        return launch_dep(d, kernel, grid, block, smem, st, std::forward<Args>(args)...);
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return cudaErrorUnknown;
    cudaEventRecord(e0, st);
    cudaError_t rc = launch(d, kernel, grid, block, smem, st, std::forward<Args>(args)...);
    cudaEventRecord(e1, st);
    std::lock_guard<std::mutex> lk(d->timing_mu);
    d->timing_ev[which].emplace_back(e0, e1);
    return rc;
}

// Select of a launch over n_slots consumer slots: tiles of one or of several passes, by the
// dock's size.
template <typename... Args>
cudaError_t launch_select(td_dock *d, uint32_t n_slots, cudaStream_t st, Args &&...args) {
    const uint32_t G = d->dv.G;
    if (sel_passes(G) > 1)
        return launch_dep(d, get_select_kernel<(int)kSelWide>, dim3(sel_tiles(G), n_slots), dim3(kSelThreads), 0, st,
                          std::forward<Args>(args)...);
    return launch_dep(d, get_select_kernel<1>, dim3(sel_tiles(G), n_slots), dim3(kSelThreads), 0, st,
                      std::forward<Args>(args)...);
}

// Finalize of a launch whose largest request may serve up to max_samples samples: one CTA per
// request, a large block when a request is large (its scans then take a quarter of the rounds).
template <typename... Args>
cudaError_t launch_finalize(td_dock *d, uint32_t n_req, uint32_t max_samples, cudaStream_t st, Args &&...args) {
    if (max_samples > kFinBigSamples)
        return launch_dep(d, get_finalize_kernel<kFinThreadsBig, false>, dim3(n_req), dim3(kFinThreadsBig), 0, st,
                          std::forward<Args>(args)...);
    return launch_dep(d, get_finalize_kernel<kFinThreads, false>, dim3(n_req), dim3(kFinThreads), 0, st,
                      std::forward<Args>(args)...);
}

// May the scan of a call run inside its finalize kernel?  The dock's groups fit one wide tile,
// every consumer of the call has one request, and no request is large.
bool scan_fits_finalize(const td_dock *d, uint32_t n_req, uint32_t n_slots, uint32_t max_samples) {
    return d->dv.G <= kSelThreads * kSelWide && n_req == n_slots && max_samples <= kFinBigSamples;
}
template <typename... Args>
cudaError_t launch_fused_finalize(td_dock *d, uint32_t n_req, cudaStream_t st, Args &&...args) {
    static_assert(kFinThreads == kSelThreads, "the fused scan is one tile of the finalize kernel's threads");
    return launch_dep(d, get_finalize_kernel<kFinThreads, true>, dim3(n_req), dim3(kFinThreads), 0, st,
                      std::forward<Args>(args)...);
}

void drop_timing(td_dock *d) {
    std::lock_guard<std::mutex> lk(d->timing_mu);
    for (auto &v : d->timing_ev) {
        for (auto &p : v) { cudaEventDestroy(p.first); cudaEventDestroy(p.second); }
        v.clear();
    }
}

}  // namespace

extern "C" {

// Eq. 1, Eq. 2 and Eq. 4 in exact integer arithmetic (128-bit intermediates, overflow = TD_EINVAL).
int td_model_bytes(const td_model *m, uint64_t *cv, uint64_t *tcv, double *tcv_dock) {
    if (!m) return TD_EINVAL;
    typedef unsigned __int128 u128;
    const u128 lim = (u128)1 << 64;
    auto mul = [&](u128 a, u128 b, bool &ok) -> u128 {
        if (a >= lim || b >= lim) { ok = false; return 0; }     // factors below 2^64: the product fits 128 bits
        const u128 p = a * b;
        if (p >= lim) ok = false;
        return p;
    };
    bool ok = true;
    const u128 samples = mul(mul(m->G, m->N, ok), m->B, ok);                 // G*N*B
    const u128 resp = mul(m->n, m->SL, ok);                                   // n*SL
    const u128 per1 = (u128)m->PL + resp + m->M;                              // Eq. 1 bracket
    const u128 per2 = 2 * (u128)m->PL + 3 * resp + 8 * (u128)m->M;            // Eq. 2 bracket
    const u128 v1 = mul(samples, per1, ok), v2 = mul(samples, per2, ok);
    if (!ok) return TD_EINVAL;
    if (cv) *cv = (uint64_t)v1;
    if (tcv) *tcv = (uint64_t)v2;
    if (tcv_dock) {
        if (m->S == 0) return TD_EINVAL;
        const u128 meta = mul(8 * ((u128)m->C + 1), m->M, ok);                // 8*(C+1)*M
        const u128 per4 = 2 * (u128)m->PL + 3 * resp + meta;
        const u128 v4 = mul(samples, per4, ok);
        if (!ok) return TD_EINVAL;
        *tcv_dock = (double)(uint64_t)v4 / (double)m->S;
    }
    return TD_OK;
}

const char *td_strerror(int code) {
    switch (code) {
        case TD_OK: return "ok";
        case TD_EINVAL: return "invalid argument";
        case TD_EWORKSPACE: return "workspace or scratch too small or misaligned";
        case TD_ECUDA: return "CUDA runtime call failed";
        case TD_ETOOLARGE: return "dock has more prompts than the fixed-scratch get supports";
        default: return "unknown error";
    }
}

int td_query_workspace(const td_config *cfg, size_t *bytes) {
    if (!bytes || !valid_config(cfg)) return TD_EINVAL;
    *bytes = make_layout(cfg).total;
    return TD_OK;
}

int td_create(const td_config *cfg, void *d_workspace, size_t bytes, td_dock **out) {
    if (!out || !d_workspace || !valid_config(cfg)) return TD_EINVAL;
    const Layout L = make_layout(cfg);
    if (bytes < L.total || (reinterpret_cast<uintptr_t>(d_workspace) & 255u)) return TD_EWORKSPACE;
    if (cudaSetDevice(cfg->device) != cudaSuccess) return TD_ECUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess) return TD_ECUDA;
    const size_t alloc_smem = put_alloc_smem_bytes(cfg->n_shards);
    if (cudaFuncSetAttribute(put_alloc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)alloc_smem) != cudaSuccess ||
        cudaFuncSetAttribute(put_alloc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)alloc_smem) != cudaSuccess ||
        cudaFuncSetAttribute(put_alloc_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)alloc_smem) != cudaSuccess)
        return TD_ECUDA;

    if (cudaFuncSetAttribute(put_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)scatter_smem_bytes()) != cudaSuccess ||
        cudaFuncSetAttribute(get_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)gather_smem_bytes(kMaxJobs, 1)) != cudaSuccess)
        return TD_ECUDA;

    td_dock *d = new (std::nothrow) td_dock();
    if (!d) return TD_EINVAL;
    d->cfg = *cfg; d->cfg.columns = nullptr; d->cfg.consumers = nullptr;
    d->device = cfg->device; d->sm_count = sms;
    d->ws = static_cast<uint8_t *>(d_workspace); d->ws_bytes = bytes;
    d->launches = 0;
    d->timing = false;
    DockView &v = d->dv;
    std::memset(&v, 0, sizeof(v));
    v.G = cfg->n_prompts; v.N = cfg->n_per_group; v.S = cfg->n_shards; v.n = v.G * v.N;
    v.ncol = cfg->n_columns; v.ncons = cfg->n_consumers;
    v.prompts_per_shard = v.G / v.S;
    v.div_shard = make_fastdiv(v.N * v.prompts_per_shard);
    v.reward_col = cfg->reward_column;
    v.claim_words = L.claim_words; v.consumed_words = L.consumed_words;
    v.spin_limit = kDefaultPollLimit;
    v.lookback_limit = kDefaultPollLimit;
    v.debug_skip_tile = 0xffffffffu;
    v.eps = (double)cfg->adv_eps;
    v.cap[1] = L.cap[1]; v.cap[2] = L.cap[2];
    uint8_t *w = d->ws;
    v.status = reinterpret_cast<uint32_t *>(w + L.status);
    for (int k = 1; k <= 2; ++k) {
        v.len[k] = reinterpret_cast<int32_t *>(w + L.len[k]);
        v.off[k] = reinterpret_cast<long long *>(w + L.off[k]);
        v.cursor[k] = reinterpret_cast<unsigned long long *>(w + L.cursor[k]);
    }
    v.claim = reinterpret_cast<uint32_t *>(w + L.claim);
    v.consumed = reinterpret_cast<uint32_t *>(w + L.consumed);
    v.errword = reinterpret_cast<uint32_t *>(w + L.errword);
    v.counters = reinterpret_cast<unsigned long long *>(w + L.counters);
    v.put_counters = reinterpret_cast<unsigned long long *>(w + L.put_counters);
    v.put_ready = reinterpret_cast<unsigned long long *>(w + L.put_ready);
    v.progress = reinterpret_cast<uint32_t *>(w + L.progress);
    for (uint32_t k = 0; k < v.ncol; ++k) {
        v.colbase[k] = w + L.col[k];
        v.col_esz[k] = (uint8_t)esize_of(cfg->columns[k].dtype);
        v.col_cls[k] = (uint8_t)cfg->columns[k].cls;
        v.col_pad[k] = cfg->columns[k].pad_bits;
    }
    for (uint32_t k = 0; k < v.ncons; ++k) {
        v.need[k] = cfg->consumers[k].need_mask;
        v.outm[k] = cfg->consumers[k].out_mask;
        v.cflags[k] = cfg->consumers[k].flags;
    }
    d->table_bytes[0] = (size_t)v.n * 4; d->table_bytes[1] = (size_t)v.n * 4; d->table_bytes[2] = (size_t)v.n * 8;
    d->table_bytes[3] = (size_t)v.S * 8; d->table_bytes[4] = (size_t)v.claim_words * 4;
    d->table_bytes[5] = (size_t)v.consumed_words * 4; d->table_bytes[6] = 0;

    int rc = cudaMemsetAsync(w + L.put_ready, 0, (size_t)kPutCounterSlots * 4 * 8, nullptr) == cudaSuccess ? TD_OK : TD_ECUDA;
    if (rc == TD_OK) rc = td_reset(d, nullptr);
    if (rc == TD_OK && cudaStreamSynchronize(nullptr) != cudaSuccess) rc = TD_ECUDA;
    if (rc != TD_OK) { delete d; return rc; }
    *out = d;
    return TD_OK;
}

int td_destroy(td_dock *dock) {
    if (dock) drop_timing(dock);
    delete dock;
    return TD_OK;
}

int td_reset(td_dock *d, void *stream) {
    TD_RANGE("td_reset");
    if (!d) return TD_EINVAL;
    const uint32_t blocks = (uint32_t)std::min<size_t>((d->dv.n + 255) / 256, (size_t)d->sm_count * 4);
    if (launch(d, reset_kernel, dim3(blocks ? blocks : 1), dim3(256), 0, (cudaStream_t)stream, d->dv) != cudaSuccess)
        return TD_ECUDA;
    return TD_OK;
}

namespace {

// Grid of a copy launch that may move up to room_bytes on the packed side: one resident wave
// at most, fewer CTAs when there is less than a minimum chunk per warp.
uint32_t copy_grid(const td_dock *d, uint64_t room_bytes) {
    const uint64_t max_blocks = (uint64_t)d->sm_count * kCopyBlocksPerSM;
    uint64_t blocks = (room_bytes / kMinChunkBytes + kCopyWarps) / kCopyWarps;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks == 0) blocks = 1;
    return (uint32_t)blocks;
}

// The slot of stream `st` in the dock's per-stream words (the scatter kernel's chunk counter, the
// word in which the alloc kernel tells it that the call's inputs are complete), or -1.  Calls
// on one stream run one after the other, so a slot per stream is never shared by two launches
// in flight.  A call that is being captured into a graph gets none: the graph may later run on
// any stream, beside anything.
int stream_slot(td_dock *d, cudaStream_t st) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) {
        cudaGetLastError();
        return -1;
    }
    std::lock_guard<std::mutex> lk(d->slot_mu);
    for (size_t i = 0; i < d->slot_stream.size(); ++i)
        if (d->slot_stream[i] == st) return (int)i;
    if (d->slot_stream.size() >= (size_t)kPutCounterSlots) return -1;
    d->slot_stream.push_back(st);
    return (int)d->slot_stream.size() - 1;
}

// One launch group: alloc and scatter (which also publishes), or, for scalar columns only, one
// publish kernel.  Items are taken in order; a column appears at most once per group, so that
// duplicate detection sees earlier items.
int put_group(td_dock *d, PutBatch &b, cudaStream_t st) {
    const DockView &v = d->dv;
    // Propose followers to the alloc kernel: an item may ride along with the latest item of its
    // length class that takes passes of its own, when it has the same entry count and not more
    // data behind it.
    int leader[3] = {-1, -1, -1};
    for (uint32_t i = 0; i < kMaxPutItems; ++i) b.follow[i] = 0;
    for (uint32_t i = 0; i < b.n_items; ++i) {
        const PutArgs &a = b.item[i];
        const uint32_t cls = v.col_cls[a.column];
        if (cls == TD_SCALAR) continue;
        const int l = leader[cls];
        if (l >= 0 && b.item[l].k == a.k && b.item[l].k_dev == a.k_dev && a.data_elems <= b.item[l].data_elems)
            b.follow[i] = (uint8_t)(l + 1);
        else
            leader[cls] = (int)i;
    }
    uint64_t ragged_bytes = 0, entries = 0;
    for (uint32_t i = 0; i < b.n_items; ++i) {
        entries += b.item[i].k;
        if (v.col_cls[b.item[i].column] != TD_SCALAR)
            ragged_bytes += b.item[i].data_elems * v.col_esz[b.item[i].column] + kMinChunkBytes;
    }
    if (entries == 0) return TD_OK;
    if (entries >= (1ull << 32)) return TD_EINVAL;
    b.work_counter = nullptr; b.ready = nullptr; b.progress = nullptr; b.seq = 0;
    if (ragged_bytes) {
        // The words the two kernels talk through carry the call's number, and numbers must grow in
        // the order the calls reach their stream: two host threads putting on one stream take
        // their number and enqueue under one lock.
        std::lock_guard<std::mutex> order(d->put_mu);
        const int slot = stream_slot(d, st);
        if (slot >= 0) {
            b.work_counter = d->dv.put_counters + slot;
            b.ready = d->dv.put_ready + 4 * (size_t)slot;
            b.seq = g_put_seq.fetch_add(1, std::memory_order_relaxed);
            // the per-class counts of allocated entries go by the order of the leader items, which is
            // only known here when no follower has to be compared with its leader on the device
            bool settled = true;
            for (uint32_t i = 0; i < b.n_items; ++i)
                if (b.follow[i]) {
                    const PutArgs &a = b.item[i], &ld = b.item[b.follow[i] - 1u];
                    settled = settled && a.idx == ld.idx && a.cu == ld.cu;
                }
            if (settled) b.progress = b.ready + 1;
        }
        ragged_bytes += entries * kPutScalarCost;              // the scalar items of the call ride along
        // entries per thread and pass of the alloc kernel: enough for the largest item in one pass, up to four
        uint32_t k_max = 0;
        for (uint32_t i = 0; i < b.n_items; ++i)
            if (v.col_cls[b.item[i].column] != TD_SCALAR) k_max = std::max(k_max, b.item[i].k);
        auto alloc_kernel = k_max <= (uint32_t)kAllocThreads ? put_alloc_kernel<1>
                            : k_max <= 2u * kAllocThreads ? put_alloc_kernel<2> : put_alloc_kernel<4>;
        if (launch_dep(d, alloc_kernel, dim3(2), dim3(kAllocThreads), put_alloc_smem_bytes(v.S), st, v, b) != cudaSuccess)
            return TD_ECUDA;
        if (launch_timed(d, 0, put_scatter_kernel, dim3(copy_grid(d, ragged_bytes)), dim3(kCopyThreads),
                         scatter_smem_bytes(), st, v, b) != cudaSuccess)
            return TD_ECUDA;
        return TD_OK;
    }
    if (launch_dep(d, put_publish_kernel, dim3((uint32_t)((entries + 255) / 256)), dim3(256), 0, st, v, b) != cudaSuccess)
        return TD_ECUDA;
    return TD_OK;
}

bool valid_put_item(const td_dock *d, const td_put_item &it) {
    if (it.column >= d->dv.ncol) return false;
    if (it.k == 0) return true;
    if (!it.d_indices || (!it.d_data && it.data_elems)) return false;
    if (d->dv.col_cls[it.column] != TD_SCALAR && !it.d_cu) return false;
    return it.data_elems < (1ull << 31);                 // cu is int32
}


uint64_t room_bytes_of(const DockView &v, uint32_t consumer, uint32_t max_samples, const td_get_out &out) {
    uint64_t bytes = 0;
    for (uint32_t k = 0; k < v.ncol; ++k)
        if (((v.outm[consumer] >> k) & 1u) && out.col[k]) {
            uint64_t room = out.col_capacity_elems[k];
            if (v.col_cls[k] == TD_SCALAR && room > max_samples) room = max_samples;
            bytes += room * v.col_esz[k] + kMinChunkBytes;
        }
    if (out.seq) bytes += out.seq_capacity_elems * v.col_esz[out.seq_prompt_col] + kMinChunkBytes;
    if (out.seq_advantages) bytes += out.seq_capacity_elems * 4u + kMinChunkBytes;
    return bytes;
}

bool wants_stream(const td_get_out &out) { return out.seq || out.seq_advantages; }
uint32_t jobs_per_req(const DockView &v, bool stream) { return v.ncol + (stream ? kSeqJobs : 0u); }

// The room a request's output buffers leave (see GetReq): by class, over the wanted columns.
void fill_room(const DockView &v, uint32_t consumer, const td_get_out &out, GetReq &rq) {
    rq.room_tok[0] = rq.room_tok[1] = rq.room_tok[2] = ~0ull;
    rq.room_rows = ~0ull;
    rq.want_classes = 0;
    for (uint32_t k = 0; k < v.ncol; ++k) {
        if (!((v.outm[consumer] >> k) & 1u) || out.col[k] == nullptr) continue;
        const uint32_t cls = v.col_cls[k];
        const uint64_t capk = out.col_capacity_elems[k];
        rq.want_classes |= 1u << cls;
        if (cls == TD_SCALAR) rq.room_tok[0] = std::min<uint64_t>(rq.room_tok[0], capk);
        else if (out.mode == TD_PACKED) rq.room_tok[cls] = std::min<uint64_t>(rq.room_tok[cls], capk);
        else {
            const uint32_t W = cls == TD_PROMPT ? out.pad_prompt_to : out.pad_response_to;
            rq.room_rows = std::min<uint64_t>(rq.room_rows, W ? capk / W : 0);
        }
    }
}

// Upper bound of what a request adds to the space the gather cuts into chunks: its output room
// plus the fixed charge of every row of every job.
uint64_t extent_bound_of(const DockView &v, uint32_t consumer, uint32_t max_samples, const td_get_out &out, uint32_t jpr) {
    const uint64_t rows = (uint64_t)std::min(max_samples / v.N, v.G) * v.N;
    return room_bytes_of(v, consumer, max_samples, out) + rows * jpr * kRowCost + (uint64_t)jpr * kJobUnit;
}

int check_get_out(const DockView &v, uint32_t consumer, uint32_t max_samples, const td_get_out *out) {
    if (!out || consumer >= v.ncons) return TD_EINVAL;
    if (max_samples / v.N == 0) return TD_EINVAL;
    if (!out->indices || !out->cu_prompt || !out->cu_response || !out->result) return TD_EINVAL;
    if (out->mode != TD_PACKED && out->mode != TD_PADDED) return TD_EINVAL;
    if (out->flags & ~(uint32_t)TD_OUT_LEFT_PAD_PROMPT) return TD_EINVAL;
    if ((v.cflags[consumer] & TD_F_ADVANTAGE) && !out->advantages) return TD_EINVAL;
    if (wants_stream(*out) && !out->cu_seq) return TD_EINVAL;
    if (out->seq) {
        const uint32_t cp = out->seq_prompt_col, cr = out->seq_response_col;
        if (cp >= v.ncol || cr >= v.ncol) return TD_EINVAL;
        if (v.col_cls[cp] != TD_PROMPT || v.col_cls[cr] != TD_RESPONSE || v.col_esz[cp] != v.col_esz[cr]) return TD_EINVAL;
        if (!((v.outm[consumer] >> cp) & 1u) || !((v.outm[consumer] >> cr) & 1u)) return TD_EINVAL;
    }
    if (out->seq_advantages && !((v.cflags[consumer] & TD_F_ADVANTAGE) && out->advantages)) return TD_EINVAL;
    return TD_OK;
}

}  // namespace

namespace {
// Items in call order, cut into launch groups of at most kMaxPutItems in which no column
// appears twice.
int put_items(td_dock *d, const PutArgs *items, uint32_t n_items, cudaStream_t st) {
    PutBatch b;
    std::memset(&b, 0, sizeof(b));
    uint32_t seen = 0;
    for (uint32_t i = 0; i < n_items; ++i) {
        const PutArgs &it = items[i];
        if (it.k == 0) continue;
        if (b.n_items == kMaxPutItems || (seen >> it.column) & 1u) {
            const int rc = put_group(d, b, st);
            if (rc != TD_OK) return rc;
            b.n_items = 0; seen = 0;
        }
        b.item[b.n_items++] = it;
        seen |= 1u << it.column;
    }
    return b.n_items ? put_group(d, b, st) : TD_OK;
}
}  // namespace

int td_put_many(td_dock *d, const td_put_item *items, uint32_t n_items, void *stream) {
    TD_RANGE("td_put_many");
    if (!d || (n_items && !items)) return TD_EINVAL;
    for (uint32_t i = 0; i < n_items; ++i)
        if (!valid_put_item(d, items[i])) return TD_EINVAL;
    std::vector<PutArgs> args(n_items);
    for (uint32_t i = 0; i < n_items; ++i) {
        const td_put_item &it = items[i];
        args[i] = PutArgs{it.column, it.k, it.d_indices, it.d_cu, static_cast<const uint8_t *>(it.d_data),
                          it.data_elems, nullptr};
    }
    return put_items(d, args.data(), n_items, (cudaStream_t)stream);
}

namespace {
// One write-back as a put item: the samples and row boundaries are the batch's, the count is
// read from its result block on the device.
int back_args(const td_dock *d, const td_get_out *batch, uint32_t max_samples, uint32_t column,
              const void *d_data, uint64_t data_elems, PutArgs *out) {
    const DockView &v = d->dv;
    if (!batch || !batch->indices || !batch->cu_prompt || !batch->cu_response || !batch->result) return TD_EINVAL;
    if (column >= v.ncol || (!d_data && data_elems) || data_elems >= (1ull << 31)) return TD_EINVAL;
    const uint32_t cls = v.col_cls[column];
    const int32_t *cu = cls == TD_PROMPT ? batch->cu_prompt : cls == TD_RESPONSE ? batch->cu_response : nullptr;
    *out = PutArgs{column, max_samples, batch->indices, cu, static_cast<const uint8_t *>(d_data), data_elems,
                   &batch->result->n_samples};
    return TD_OK;
}
}  // namespace

int td_put_back(td_dock *d, const td_get_out *batch, uint32_t max_samples, const td_back_item *items,
                uint32_t n_items, void *stream) {
    TD_RANGE("td_put_back");
    if (!d || !batch || (n_items && !items)) return TD_EINVAL;
    std::vector<PutArgs> args(n_items);
    for (uint32_t i = 0; i < n_items; ++i) {
        const int rc = back_args(d, batch, max_samples, items[i].column, items[i].d_data, items[i].data_elems, &args[i]);
        if (rc != TD_OK) return rc;
    }
    return put_items(d, args.data(), n_items, (cudaStream_t)stream);
}

int td_put_back_many(td_dock *d, const td_back_req *reqs, uint32_t n_reqs, void *stream) {
    TD_RANGE("td_put_back_many");
    if (!d || (n_reqs && !reqs)) return TD_EINVAL;
    std::vector<PutArgs> args(n_reqs);
    for (uint32_t i = 0; i < n_reqs; ++i) {
        const int rc = back_args(d, reqs[i].batch, reqs[i].max_samples, reqs[i].column, reqs[i].d_data,
                                 reqs[i].data_elems, &args[i]);
        if (rc != TD_OK) return rc;
    }
    return put_items(d, args.data(), n_reqs, (cudaStream_t)stream);
}

int td_put(td_dock *d, uint32_t column, const int32_t *d_indices, uint32_t k, const int32_t *d_cu,
           const void *d_data, uint64_t data_elems, void *stream) {
    const td_put_item it{column, k, d_indices, d_cu, d_data, data_elems};
    return td_put_many(d, &it, 1, stream);
}

size_t td_get_scratch_bytes(const td_dock *d) {
    return d ? sel_scratch_bytes(d->dv.G) : 0;
}

namespace {
// One get with its scan scratch at `scratch` (checked by the caller): select, finalize, gather,
// or finalize and gather where the scan fits the finalize kernel.
int get_one(td_dock *d, uint32_t consumer, uint32_t max_samples, const td_get_out *out, void *scratch,
            cudaStream_t st) {
    const DockView &v = d->dv;
    const uint32_t m = max_samples / v.N;
    GetInline one;
    std::memset(&one, 0, sizeof(one));
    one.req.out = *out;
    one.req.consumer = consumer;
    one.req.max_groups = m < v.G ? m : v.G;
    one.req.rank_base = 0;
    one.req.cslot = 0;
    fill_room(v, consumer, *out, one.req);
    one.cs.consumer = consumer;
    one.cs.max_groups = one.req.max_groups;
    one.cs.scratch = scratch;
    const uint32_t seq = g_seq.fetch_add(1, std::memory_order_relaxed);
    const uint32_t jpr = jobs_per_req(v, wants_stream(*out));
    if (extent_bound_of(v, consumer, max_samples, *out, jpr) >= kMaxLaunchExtent) return TD_EINVAL;

    // word 1 of the scan scratch is the gather's chunk counter
    unsigned long long *counter = static_cast<unsigned long long *>(scratch) + 1;
    if (scan_fits_finalize(d, 1u, 1u, one.req.max_groups * v.N)) {
        if (launch_fused_finalize(d, 1u, st, v, one, (const GetReq *)nullptr, (const ConsumerSlot *)nullptr, seq, counter,
                                  (JobSize *)nullptr, jpr, (uint8_t *)nullptr) != cudaSuccess) return TD_ECUDA;
    } else {
        if (launch_select(d, 1u, st, v, one, (const ConsumerSlot *)nullptr, seq) != cudaSuccess) return TD_ECUDA;
        if (launch_finalize(d, 1u, one.req.max_groups * v.N, st, v, one, (const GetReq *)nullptr,
                            (const ConsumerSlot *)nullptr, seq, counter, (JobSize *)nullptr, jpr, (uint8_t *)nullptr) !=
            cudaSuccess) return TD_ECUDA;
    }
    const uint32_t blocks = copy_grid(d, room_bytes_of(v, consumer, max_samples, *out));
    if (launch_timed(d, 1, get_gather_kernel, dim3(blocks), dim3(kCopyThreads), gather_smem_bytes(1, jpr), st, v, one,
                     (const GetReq *)nullptr, 1u, counter, (const JobSize *)nullptr, jpr, make_fastdiv(jpr),
                     (const ConsumerSlot *)nullptr, 1u) != cudaSuccess) return TD_ECUDA;
    return TD_OK;
}
}  // namespace

int td_get(td_dock *d, uint32_t consumer, uint32_t max_samples, const td_get_out *out, void *stream) {
    TD_RANGE("td_get");
    if (!d) return TD_EINVAL;
    const DockView &v = d->dv;
    const int chk = check_get_out(v, consumer, max_samples, out);
    if (chk != TD_OK) return chk;
    if (!out->scratch || (reinterpret_cast<uintptr_t>(out->scratch) & 15u) ||
        out->scratch_bytes < sel_scratch_bytes(v.G))
        return TD_EWORKSPACE;
    return get_one(d, consumer, max_samples, out, out->scratch, (cudaStream_t)stream);
}

// ---- a get whose scan scratch is a fixed array inside the library ----
// For callers that have nowhere to take scratch memory from: code running where device memory
// may not be allocated (inside a serving loop with a frozen memory pool, in a plug-in that was
// handed only its input and output buffers, under a memory budget that is already spent).
// td_get makes such a caller supply td_get_scratch_bytes() of zero-filled device memory; this
// variant keeps that scratch in the array below instead, which every device that loads the
// library holds (kStaticScratchBytes, about 65 KB) until the process exits.
constexpr uint32_t kStaticMaxGroups = 16384;          // docks with more prompts are refused
constexpr size_t kStaticScratchBytes = sel_scratch_bytes(kStaticMaxGroups);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void *g_static_ptr[kMaxDevices] = {};                 // device address of g_static_scratch, per device

// In host code the array's name is only a handle: the device address has to be asked for, once
// per device, with that device current.
int static_scratch_address(int device, void **out) {
    if (device < 0 || device >= kMaxDevices) return TD_EINVAL;
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_static_ptr[device]) {
        int cur = -1;
        if (cudaGetDevice(&cur) != cudaSuccess) return TD_ECUDA;
        if (cur != device && cudaSetDevice(device) != cudaSuccess) return TD_ECUDA;
        void *p = nullptr;
        const cudaError_t rc = cudaGetSymbolAddress(&p, g_static_scratch);
        if (cur != device) cudaSetDevice(cur);
        if (rc != cudaSuccess || !p) return TD_ECUDA;
        g_static_ptr[device] = p;
    }
    *out = g_static_ptr[device];
    return TD_OK;
}
}  // namespace

int td_get_static(td_dock *d, uint32_t consumer, uint32_t max_samples, const td_get_out *out, void *stream) {
    TD_RANGE("td_get_static");
    if (!d) return TD_EINVAL;
    const DockView &v = d->dv;
    const int chk = check_get_out(v, consumer, max_samples, out);
    if (chk != TD_OK) return chk;
    if (v.G > kStaticMaxGroups || sel_scratch_bytes(v.G) > kStaticScratchBytes) return TD_ETOOLARGE;
    void *scratch = nullptr;
    const int rc = static_scratch_address(d->device, &scratch);
    if (rc != TD_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // The array still holds what the last call left.  The scan tags what it writes with the
    // call's sequence number, but the ticket and the tile descriptors are cleared all the same,
    // so that nothing here depends on what ran before.
    if (cudaMemsetAsync(scratch, 0, (2 + (size_t)sel_tiles(v.G)) * 8, st) != cudaSuccess) return TD_ECUDA;
    return get_one(d, consumer, max_samples, out, scratch, st);
}

// ---- plans: many gets served by one call ----
struct td_plan {
    td_dock *dock;
    uint32_t n_req, n_slots;
    GetReq *d_reqs;
    ConsumerSlot *d_slots;
    uint64_t room_bytes;
    uint32_t jobs_per_req;                // columns, plus the stream's jobs when a request wants it
    uint32_t max_req_samples;             // the largest request, in samples
    size_t meta_total;                    // bytes of the staging buffer td_get_many_host may be given
    uint8_t *h_meta;                      // its pinned host mirror, allocated by the first call that uses it
    unsigned long long *d_counter;        // the gather's chunk counter: word 1 of slot 0's scan scratch
    JobSize *d_job_sizes;                 // [n_req][n_columns] output bytes and rows, written by the finalize kernel
    std::vector<uint8_t> host_image;      // what was uploaded; kept until the plan dies
};

size_t td_plan_bytes(const td_dock *d, uint32_t n_req) {
    if (!d || n_req == 0) return 0;
    const size_t slots = d->dv.ncons;
    return align_up_sz((size_t)n_req * sizeof(GetReq), 256) + align_up_sz(slots * sizeof(ConsumerSlot), 256) +
           slots * align_up_sz(sel_scratch_bytes(d->dv.G), 256) +
           align_up_sz((size_t)n_req * (d->dv.ncol + kSeqJobs) * sizeof(JobSize), 256);
}

int td_plan_create(td_dock *d, const td_get_req *reqs, uint32_t n_req, void *d_plan, size_t plan_bytes,
                   void *stream, td_plan **out) {
    if (!d || !reqs || !out || n_req == 0) return TD_EINVAL;
    const DockView &v = d->dv;
    bool stream_wanted = false;
    for (uint32_t q = 0; q < n_req; ++q) stream_wanted |= wants_stream(reqs[q].out);
    const uint32_t jpr = jobs_per_req(v, stream_wanted);
    if ((uint64_t)n_req * jpr > (uint64_t)kMaxJobs) return TD_EINVAL;
    if (!d_plan || (reinterpret_cast<uintptr_t>(d_plan) & 255u) || plan_bytes < td_plan_bytes(d, n_req))
        return TD_EWORKSPACE;
    for (uint32_t q = 0; q < n_req; ++q) {
        const int chk = check_get_out(v, reqs[q].consumer, reqs[q].max_samples, &reqs[q].out);
        if (chk != TD_OK) return chk;
    }
    td_plan *p = new (std::nothrow) td_plan();
    if (!p) return TD_EINVAL;
    p->dock = d; p->n_req = n_req; p->jobs_per_req = jpr;
    p->meta_total = 0; p->h_meta = nullptr; p->max_req_samples = 0;
    const size_t off_slots = align_up_sz((size_t)n_req * sizeof(GetReq), 256);
    const size_t off_scratch = off_slots + align_up_sz((size_t)v.ncons * sizeof(ConsumerSlot), 256);
    const size_t scratch_each = align_up_sz(sel_scratch_bytes(v.G), 256);
    uint8_t *base = static_cast<uint8_t *>(d_plan);
    p->d_reqs = reinterpret_cast<GetReq *>(base);
    p->d_slots = reinterpret_cast<ConsumerSlot *>(base + off_slots);
    p->host_image.assign(off_scratch, 0);
    GetReq *hr = reinterpret_cast<GetReq *>(p->host_image.data());
    ConsumerSlot *hs = reinterpret_cast<ConsumerSlot *>(p->host_image.data() + off_slots);
    // consumer slots in order of first appearance; requests of one consumer share its candidates
    int slot_of[32];
    for (int &x : slot_of) x = -1;
    uint32_t n_slots = 0;
    uint64_t room = 0, extent = 0;
    for (uint32_t q = 0; q < n_req; ++q) {
        extent += extent_bound_of(v, reqs[q].consumer, reqs[q].max_samples, reqs[q].out, jpr);
        if (extent >= kMaxLaunchExtent) { delete p; return TD_EINVAL; }      // more than one launch can address
        const uint32_t c = reqs[q].consumer;
        if (slot_of[c] < 0) {
            slot_of[c] = (int)n_slots;
            hs[n_slots].consumer = c; hs[n_slots].max_groups = 0;
            hs[n_slots].scratch = base + off_scratch + (size_t)n_slots * scratch_each;
            ++n_slots;
        }
        ConsumerSlot &cs = hs[slot_of[c]];
        const uint32_t m = reqs[q].max_samples / v.N;
        hr[q].out = reqs[q].out;
        hr[q].consumer = c;
        hr[q].rank_base = cs.max_groups;
        hr[q].max_groups = m;
        hr[q].cslot = (uint32_t)slot_of[c];
        hr[q].meta_samples = std::min(m, v.G) * v.N;
        fill_room(v, c, reqs[q].out, hr[q]);
        hr[q].meta_off = p->meta_total;
        p->meta_total += align_up_sz(meta_bytes(hr[q].meta_samples), 16);
        const uint64_t sum = (uint64_t)cs.max_groups + m;
        cs.max_groups = sum > v.G ? v.G : (uint32_t)sum;
        if (hr[q].rank_base > v.G) hr[q].rank_base = v.G;
        room += room_bytes_of(v, c, reqs[q].max_samples, reqs[q].out);
        p->max_req_samples = std::max(p->max_req_samples, std::min(m, v.G) * v.N);
    }
    p->n_slots = n_slots;
    p->d_counter = reinterpret_cast<unsigned long long *>(base + off_scratch) + 1;
    p->d_job_sizes = reinterpret_cast<JobSize *>(base + off_scratch + (size_t)v.ncons * scratch_each);
    p->room_bytes = room;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(base + off_scratch, 0, (size_t)v.ncons * scratch_each, st) != cudaSuccess ||
        cudaMemcpyAsync(base, p->host_image.data(), off_scratch, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        delete p;
        return TD_ECUDA;
    }
    *out = p;
    return TD_OK;
}

int td_plan_destroy(td_plan *p) {
    if (p && p->h_meta) cudaFreeHost(p->h_meta);
    delete p;
    return TD_OK;
}

namespace {
int get_many(td_dock *d, td_plan *p, uint8_t *d_meta, void *stream);
}
int td_get_many(td_dock *d, td_plan *p, void *stream) {
    TD_RANGE("td_get_many"); return get_many(d, p, nullptr, stream); }

namespace {
// d_meta: staging buffer for the second copy of the requests' small outputs, or nullptr.
int get_many(td_dock *d, td_plan *p, uint8_t *d_meta, void *stream) {
    if (!d || !p || p->dock != d) return TD_EINVAL;
    const DockView &v = d->dv;
    cudaStream_t st = (cudaStream_t)stream;
    GetInline none;
    std::memset(&none, 0, sizeof(none));
    const uint32_t seq = g_seq.fetch_add(1, std::memory_order_relaxed);
    if (scan_fits_finalize(d, p->n_req, p->n_slots, p->max_req_samples)) {
        if (launch_fused_finalize(d, p->n_req, st, v, none, (const GetReq *)p->d_reqs, (const ConsumerSlot *)p->d_slots, seq,
                                  p->d_counter, p->d_job_sizes, p->jobs_per_req, d_meta) != cudaSuccess) return TD_ECUDA;
    } else {
        if (launch_select(d, p->n_slots, st, v, none, (const ConsumerSlot *)p->d_slots, seq) != cudaSuccess) return TD_ECUDA;
        if (launch_finalize(d, p->n_req, p->max_req_samples, st, v, none, (const GetReq *)p->d_reqs,
                            (const ConsumerSlot *)p->d_slots, seq, p->d_counter, p->d_job_sizes, p->jobs_per_req, d_meta) !=
            cudaSuccess) return TD_ECUDA;
    }
    if (launch_timed(d, 1, get_gather_kernel, dim3(copy_grid(d, p->room_bytes)), dim3(kCopyThreads),
                     gather_smem_bytes(p->n_req, p->jobs_per_req), st, v, none,
                     (const GetReq *)p->d_reqs, p->n_req, p->d_counter, (const JobSize *)p->d_job_sizes,
                     p->jobs_per_req, make_fastdiv(p->jobs_per_req), (const ConsumerSlot *)p->d_slots,
                     p->n_slots) != cudaSuccess) return TD_ECUDA;
    return TD_OK;
}
}  // namespace

int td_status(td_dock *d, td_stats *host_out, void *stream) {
    if (!d || !host_out) return TD_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long cnt[CNT_TOTAL];
    uint32_t err = 0;
    if (cudaMemcpyAsync(cnt, d->dv.counters, sizeof(cnt), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TD_ECUDA;
    if (cudaMemcpyAsync(&err, d->dv.errword, sizeof(err), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TD_ECUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return TD_ECUDA;
    std::memset(host_out, 0, sizeof(*host_out));
    for (int i = 0; i < 32; ++i) {
        host_out->put_accepted[i] = cnt[CNT_PUT_ACCEPTED + i];
        host_out->got_samples[i] = cnt[CNT_GOT_SAMPLES + i];
        host_out->got_tokens[i] = cnt[CNT_GOT_TOKENS + i];
    }
    host_out->n_oob = cnt[CNT_OOB]; host_out->n_dup = cnt[CNT_DUP];
    host_out->n_len_mismatch = cnt[CNT_MISMATCH]; host_out->n_arena_full = cnt[CNT_FULL];
    host_out->n_truncated = cnt[CNT_TRUNC]; host_out->n_bad_length = cnt[CNT_BADLEN];
    host_out->n_claim_conflicts = cnt[CNT_CONFLICT]; host_out->n_lookback_timeouts = cnt[CNT_TIMEOUT];
    host_out->error_word = err & ~kErrIrregularCu;          // the internal bit is not a condition of the ABI
    return TD_OK;
}

// Test hook: how long a scan tile waits for the tiles ahead of it, and one tile that never shows
// up.  Only the look-back wait is touched; the waits on staged copies keep their limit.
int td_debug_lookback(td_dock *d, uint32_t poll_limit, uint32_t skip_tile) {
    if (!d) return TD_EINVAL;
    d->dv.lookback_limit = poll_limit ? poll_limit : kDefaultPollLimit;
    d->dv.debug_skip_tile = skip_tile;
    return TD_OK;
}

int td_debug_table(const td_dock *d, int which, uint32_t index, void **d_ptr, size_t *bytes) {
    if (!d || !d_ptr || !bytes) return TD_EINVAL;
    const DockView &v = d->dv;
    switch (which) {
        case 0: *d_ptr = v.status; *bytes = (size_t)v.n * 4; return TD_OK;
        case 1: if (index < 1 || index > 2) return TD_EINVAL; *d_ptr = v.len[index]; *bytes = (size_t)v.n * 4; return TD_OK;
        case 2: if (index < 1 || index > 2) return TD_EINVAL; *d_ptr = v.off[index]; *bytes = (size_t)v.n * 8; return TD_OK;
        case 3: if (index < 1 || index > 2) return TD_EINVAL; *d_ptr = v.cursor[index]; *bytes = (size_t)v.S * 8; return TD_OK;
        case 4: if (index >= v.ncons) return TD_EINVAL; *d_ptr = v.claim + (size_t)index * v.claim_words; *bytes = (size_t)v.claim_words * 4; return TD_OK;
        case 5: if (index >= v.ncons) return TD_EINVAL; *d_ptr = v.consumed + (size_t)index * v.consumed_words; *bytes = (size_t)v.consumed_words * 4; return TD_OK;
        case 6: {
            if (index >= v.ncol) return TD_EINVAL;
            *d_ptr = v.colbase[index];
            const uint32_t cls = v.col_cls[index];
            *bytes = cls == TD_SCALAR ? (size_t)v.n * v.col_esz[index] : (size_t)v.S * v.cap[cls] * v.col_esz[index];
            return TD_OK;
        }
        default: return TD_EINVAL;
    }
}

uint64_t td_launch_count(const td_dock *d) { return d ? d->launches.load() : 0; }

// Self-check of the dock's bookkeeping: copies the tables to the host and tests what must hold
// between any two calls, whatever was put or served.  Synchronises the stream.
int td_debug_validate(td_dock *d, void *stream, td_validate_report *rep) {
    if (!d || !rep) return TD_EINVAL;
    std::memset(rep, 0, sizeof(*rep));
    const DockView &v = d->dv;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t n = v.n;
    std::vector<uint32_t> status(n), claim((size_t)v.ncons * v.claim_words), consumed((size_t)v.ncons * v.consumed_words);
    std::vector<int32_t> len[3];
    std::vector<long long> off[3];
    std::vector<unsigned long long> cursor[3], counters(CNT_TOTAL);
    auto d2h = [&](void *dst, const void *src, size_t bytes) {
        return bytes == 0 || cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    };
    bool ok = d2h(status.data(), v.status, n * 4) && d2h(claim.data(), v.claim, claim.size() * 4) &&
              d2h(consumed.data(), v.consumed, consumed.size() * 4) && d2h(counters.data(), v.counters, CNT_TOTAL * 8);
    for (int L = 1; L <= 2 && ok; ++L) {
        len[L].resize(n); off[L].resize(n); cursor[L].resize(v.S);
        ok = d2h(len[L].data(), v.len[L], n * 4) && d2h(off[L].data(), v.off[L], n * 8) &&
             d2h(cursor[L].data(), v.cursor[L], (size_t)v.S * 8);
    }
    if (!ok || cudaStreamSynchronize(st) != cudaSuccess) return TD_ECUDA;

    auto fail = [&](uint32_t bit, uint64_t sample) {
        if (!rep->violations) rep->first_sample = sample;
        rep->violations |= bit;
    };
    uint32_t ragged_mask[3] = {0, 0, 0}, all_mask = 0;
    for (uint32_t k = 0; k < v.ncol; ++k) { ragged_mask[v.col_cls[k]] |= 1u << k; all_mask |= 1u << k; }
    const uint32_t per_shard = v.N * v.prompts_per_shard;
    for (int L = 1; L <= 2; ++L) {
        // rows of a shard, sorted by where they start, must not overlap and must end below the cursor
        std::vector<std::vector<std::pair<long long, long long>>> rows(v.S);
        for (size_t s = 0; s < n; ++s) {
            const bool has_len = len[L][s] >= 0, has_off = off[L][s] >= 0;
            if ((status[s] & ragged_mask[L]) && !(has_len && has_off)) fail(TD_BAD_STORED_WITHOUT_ROW, s);
            if (has_off && !has_len) fail(TD_BAD_STORED_WITHOUT_ROW, s);
            if (has_len && has_off) {
                const long long room = ((long long)len[L][s] + (kRowAlign - 1)) / kRowAlign * kRowAlign;
                rows[s / per_shard].emplace_back(off[L][s], off[L][s] + room);
                if ((off[L][s] % kRowAlign) != 0) fail(TD_BAD_ROW_PLACEMENT, s);
            }
        }
        for (uint32_t sh = 0; sh < v.S; ++sh) {
            auto &r = rows[sh];
            std::sort(r.begin(), r.end());
            long long end = 0, used = 0;
            for (auto &iv : r) {
                if (iv.first < end && iv.second > iv.first) fail(TD_BAD_ROW_OVERLAP, sh);
                end = std::max(end, iv.second);
                used += iv.second - iv.first;
            }
            if ((unsigned long long)end > cursor[L][sh] || cursor[L][sh] > v.cap[L]) fail(TD_BAD_ROW_PLACEMENT, sh);
            rep->arena_elems_used[L] += (uint64_t)used;
        }
    }
    for (size_t s = 0; s < n; ++s)
        if (status[s] & ~all_mask) fail(TD_BAD_STATUS_BITS, s);
    for (uint32_t k = 0; k < v.ncol; ++k) {
        uint64_t have = 0;
        for (size_t s = 0; s < n; ++s) have += (status[s] >> k) & 1u;
        if (have != counters[CNT_PUT_ACCEPTED + k]) fail(TD_BAD_COUNTERS, k);
        rep->stored[k] = have;
    }
    for (uint32_t c = 0; c < v.ncons; ++c) {
        const uint32_t *cl = &claim[(size_t)c * v.claim_words], *co = &consumed[(size_t)c * v.consumed_words];
        uint64_t served = 0;
        for (uint32_t g = 0; g < v.G; ++g) {
            const bool claimed = (cl[g >> 5] >> (g & 31)) & 1u;
            for (uint32_t j = 0; j < v.N; ++j) {
                const size_t s = (size_t)g * v.N + j;
                const bool done = (co[s >> 5] >> (s & 31)) & 1u;
                served += done;
                if (done && !claimed) fail(TD_BAD_SERVED_UNCLAIMED, s);
                // a sample that was served had everything its consumer needs
                if (done && (status[s] & v.need[c]) != v.need[c]) fail(TD_BAD_SERVED_NOT_READY, s);
            }
        }
        if (served != counters[CNT_GOT_SAMPLES + c]) fail(TD_BAD_COUNTERS, c);
        rep->served[c] = served;
    }
    return TD_OK;
}

int td_kernel_timing(td_dock *d, int enable) {
    if (!d) return TD_EINVAL;
    drop_timing(d);
    d->timing = enable != 0;
    return TD_OK;
}

int td_kernel_timing_read(td_dock *d, int which, uint64_t *launches, double *total_ms) {
    if (!d || which < 0 || which > 1 || !launches || !total_ms) return TD_EINVAL;
    std::lock_guard<std::mutex> lk(d->timing_mu);
    double sum = 0.0;
    for (auto &p : d->timing_ev[which]) {
        if (cudaEventSynchronize(p.second) != cudaSuccess) return TD_ECUDA;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, p.first, p.second) != cudaSuccess) return TD_ECUDA;
        sum += ms;
    }
    *launches = d->timing_ev[which].size();
    *total_ms = sum;
    return TD_OK;
}

// ---- host-buffer variants: the same put / get with the copies across the bus included ----
size_t td_put_host_stage_bytes(const td_dock *d, uint32_t column, uint32_t k, uint64_t data_elems) {
    if (!d || column >= d->dv.ncol) return 0;
    return align_up_sz((size_t)k * 4, 256) + align_up_sz(((size_t)k + 1) * 4, 256) +
           align_up_sz((size_t)data_elems * d->dv.col_esz[column], 256);
}

int td_put_host(td_dock *d, uint32_t column, const int32_t *h_indices, uint32_t k, const int32_t *h_cu,
                const void *h_data, uint64_t data_elems, void *d_stage, size_t stage_bytes, void *stream) {
    TD_RANGE("td_put_host");
    if (!d || column >= d->dv.ncol) return TD_EINVAL;
    if (k == 0) return TD_OK;
    if (!h_indices || (!h_data && data_elems) || !d_stage) return TD_EINVAL;
    const bool ragged = d->dv.col_cls[column] != TD_SCALAR;
    if (ragged && !h_cu) return TD_EINVAL;
    if ((reinterpret_cast<uintptr_t>(d_stage) & 255u) || stage_bytes < td_put_host_stage_bytes(d, column, k, data_elems))
        return TD_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *p = static_cast<uint8_t *>(d_stage);
    int32_t *d_idx = reinterpret_cast<int32_t *>(p);
    int32_t *d_cu = reinterpret_cast<int32_t *>(p + align_up_sz((size_t)k * 4, 256));
    uint8_t *d_dat = reinterpret_cast<uint8_t *>(d_cu) + align_up_sz(((size_t)k + 1) * 4, 256);
    const size_t esz = d->dv.col_esz[column];
    if (cudaMemcpyAsync(d_idx, h_indices, (size_t)k * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return TD_ECUDA;
    if (ragged && cudaMemcpyAsync(d_cu, h_cu, ((size_t)k + 1) * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return TD_ECUDA;
    if (data_elems && cudaMemcpyAsync(d_dat, h_data, (size_t)data_elems * esz, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return TD_ECUDA;
    return td_put(d, column, d_idx, k, ragged ? d_cu : nullptr, d_dat, data_elems, stream);
}

namespace {
// Device -> host copies of the valid part of one served batch, sizes taken from its result block
// (already on the host).  Enqueues only.
int copy_batch_to_host(const DockView &v, uint32_t consumer, const td_get_out *dev_out, const td_get_out *host_out,
                       const td_result *res, cudaStream_t st) {
    const size_t n = res->n_samples;
    // the transfers wanted, in order; neighbours that continue each other on both sides go as one
    struct Piece { uint8_t *dst; const uint8_t *src; size_t bytes; };
    Piece todo[8 + 2 * kMaxColumns] = {};
    int n_todo = 0;
    auto d2h = [&](void *dst, const void *src, size_t bytes) {
        if (!dst || !src || bytes == 0) return;
        Piece p{static_cast<uint8_t *>(dst), static_cast<const uint8_t *>(src), bytes};
        if (n_todo && todo[n_todo - 1].dst + todo[n_todo - 1].bytes == p.dst &&
            todo[n_todo - 1].src + todo[n_todo - 1].bytes == p.src)
            todo[n_todo - 1].bytes += bytes;
        else
            todo[n_todo++] = p;
    };
    d2h(host_out->indices, dev_out->indices, n * 4);
    d2h(host_out->cu_prompt, dev_out->cu_prompt, (n + 1) * 4);
    d2h(host_out->cu_response, dev_out->cu_response, (n + 1) * 4);
    d2h(host_out->cu_seq, dev_out->cu_seq, (n + 1) * 4);
    d2h(host_out->advantages, dev_out->advantages, n * 4);
    for (uint32_t k = 0; k < v.ncol; ++k) {
        if (!((v.outm[consumer] >> k) & 1u) || !dev_out->col[k] || !host_out->col[k]) continue;
        const uint32_t cls = v.col_cls[k];
        size_t elems;
        if (cls == TD_SCALAR) elems = n;
        else if (dev_out->mode == TD_PACKED) elems = cls == TD_PROMPT ? res->prompt_tokens : res->response_tokens;
        else elems = n * (size_t)(cls == TD_PROMPT ? dev_out->pad_prompt_to : dev_out->pad_response_to);
        if (elems > host_out->col_capacity_elems[k]) return TD_EINVAL;
        d2h(host_out->col[k], dev_out->col[k], elems * v.col_esz[k]);
    }
    if (dev_out->seq && host_out->seq) {
        const size_t elems = res->prompt_tokens + res->response_tokens;
        if (elems > host_out->seq_capacity_elems) return TD_EINVAL;
        d2h(host_out->seq, dev_out->seq, elems * v.col_esz[dev_out->seq_prompt_col]);
    }
    if (dev_out->seq_advantages && host_out->seq_advantages) {
        const size_t elems = res->prompt_tokens + res->response_tokens;
        if (elems > host_out->seq_capacity_elems) return TD_EINVAL;
        d2h(host_out->seq_advantages, dev_out->seq_advantages, elems * 4);
    }
    for (int i = 0; i < n_todo; ++i)
        if (cudaMemcpyAsync(todo[i].dst, todo[i].src, todo[i].bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return TD_ECUDA;
    return TD_OK;
}
}  // namespace

int td_get_host(td_dock *d, uint32_t consumer, uint32_t max_samples, const td_get_out *dev_out,
                const td_get_out *host_out, void *stream) {
    TD_RANGE("td_get_host");
    if (!d || !dev_out || !host_out || !host_out->result || !host_out->indices) return TD_EINVAL;
    const int rc = td_get(d, consumer, max_samples, dev_out, stream);
    if (rc != TD_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    td_result *res = host_out->result;
    if (cudaMemcpyAsync(res, dev_out->result, sizeof(td_result), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TD_ECUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return TD_ECUDA;
    const int rc2 = copy_batch_to_host(d->dv, consumer, dev_out, host_out, res, st);
    if (rc2 != TD_OK) return rc2;
    if (cudaStreamSynchronize(st) != cudaSuccess) return TD_ECUDA;
    return TD_OK;
}

size_t td_get_many_host_stage_bytes(const td_plan *p) { return p ? p->meta_total : 0; }

int td_get_many_host(td_dock *d, td_plan *p, const td_get_out *host_outs, uint32_t n_req, void *d_stage,
                     size_t stage_bytes, void *stream) {
    TD_RANGE("td_get_many_host");
    if (!d || !p || p->dock != d || !host_outs || n_req != p->n_req) return TD_EINVAL;
    for (uint32_t q = 0; q < n_req; ++q)
        if (!host_outs[q].result || !host_outs[q].indices) return TD_EINVAL;
    if (d_stage && ((reinterpret_cast<uintptr_t>(d_stage) & 15u) || stage_bytes < p->meta_total)) return TD_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const GetReq *reqs = reinterpret_cast<const GetReq *>(p->host_image.data());     // the plan as uploaded
    if (d_stage && !p->h_meta &&
        cudaHostAlloc(reinterpret_cast<void **>(&p->h_meta), p->meta_total, cudaHostAllocDefault) != cudaSuccess)
        return TD_ECUDA;
    const int rc = get_many(d, p, static_cast<uint8_t *>(d_stage), stream);
    if (rc != TD_OK) return rc;
    if (d_stage) {
        // one transfer brings every request's result block, indices, cu_seqlens and advantages
        if (cudaMemcpyAsync(p->h_meta, d_stage, p->meta_total, cudaMemcpyDeviceToHost, st) != cudaSuccess) return TD_ECUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return TD_ECUDA;
        for (uint32_t q = 0; q < n_req; ++q) {
            const MetaView mv = meta_view(p->h_meta + reqs[q].meta_off, reqs[q].meta_samples);
            const td_get_out &h = host_outs[q];
            *h.result = *mv.result;
            const size_t n = mv.result->n_samples;
            std::memcpy(h.indices, mv.indices, n * 4);
            if (h.cu_prompt) std::memcpy(h.cu_prompt, mv.cu_prompt, (n + 1) * 4);
            if (h.cu_response) std::memcpy(h.cu_response, mv.cu_response, (n + 1) * 4);
            if (h.cu_seq) std::memcpy(h.cu_seq, mv.cu_seq, (n + 1) * 4);
            if (h.advantages && (d->dv.cflags[reqs[q].consumer] & TD_F_ADVANTAGE))
                std::memcpy(h.advantages, mv.advantages, n * 4);
            td_get_out payload_only = h;      // what is left to copy from the device: the columns
            payload_only.indices = nullptr; payload_only.cu_prompt = nullptr; payload_only.cu_response = nullptr;
            payload_only.cu_seq = nullptr; payload_only.advantages = nullptr;
            const int rc2 = copy_batch_to_host(d->dv, reqs[q].consumer, &reqs[q].out, &payload_only, h.result, st);
            if (rc2 != TD_OK) return rc2;
        }
    } else {
        for (uint32_t q = 0; q < n_req; ++q)
            if (cudaMemcpyAsync(host_outs[q].result, reqs[q].out.result, sizeof(td_result), cudaMemcpyDeviceToHost, st) !=
                cudaSuccess) return TD_ECUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return TD_ECUDA;
        for (uint32_t q = 0; q < n_req; ++q) {
            const int rc2 = copy_batch_to_host(d->dv, reqs[q].consumer, &reqs[q].out, &host_outs[q], host_outs[q].result, st);
            if (rc2 != TD_OK) return rc2;
        }
    }
    if (cudaStreamSynchronize(st) != cudaSuccess) return TD_ECUDA;
    return TD_OK;
}

int td_put_many_host(td_dock *d, const td_put_item *h_items, uint32_t n_items, void *d_stage, size_t stage_bytes,
                     void *stream) {
    TD_RANGE("td_put_many_host");
    if (!d || (n_items && !h_items)) return TD_EINVAL;
    if (n_items == 0) return TD_OK;
    if (!d_stage || (reinterpret_cast<uintptr_t>(d_stage) & 255u)) return TD_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    std::vector<td_put_item> dev(h_items, h_items + n_items);
    uint8_t *p = static_cast<uint8_t *>(d_stage);
    size_t used = 0;
    for (uint32_t i = 0; i < n_items; ++i) {
        const td_put_item &h = h_items[i];
        if (h.column >= d->dv.ncol) return TD_EINVAL;
        if (h.k == 0) continue;
        const bool ragged = d->dv.col_cls[h.column] != TD_SCALAR;
        if (!h.d_indices || (!h.d_data && h.data_elems) || (ragged && !h.d_cu)) return TD_EINVAL;
        const size_t need = td_put_host_stage_bytes(d, h.column, h.k, h.data_elems);
        if (used + need > stage_bytes) return TD_EWORKSPACE;
        int32_t *d_idx = reinterpret_cast<int32_t *>(p + used);
        int32_t *d_cu = reinterpret_cast<int32_t *>(p + used + align_up_sz((size_t)h.k * 4, 256));
        uint8_t *d_dat = reinterpret_cast<uint8_t *>(d_cu) + align_up_sz(((size_t)h.k + 1) * 4, 256);
        used += need;
        const size_t esz = d->dv.col_esz[h.column];
        // the columns of a record share their index array and, within a length class, their cu
        // array: what an earlier item of the call already brought over is used again
        for (uint32_t e = 0; e < i; ++e) {
            if (h_items[e].k != h.k) continue;
            if (h_items[e].d_indices == h.d_indices) d_idx = const_cast<int32_t *>(dev[e].d_indices);
            if (ragged && h_items[e].d_cu == h.d_cu && dev[e].d_cu) d_cu = const_cast<int32_t *>(dev[e].d_cu);
        }
        if (d_idx == reinterpret_cast<int32_t *>(p + used - need) &&
            cudaMemcpyAsync(d_idx, h.d_indices, (size_t)h.k * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return TD_ECUDA;
        if (ragged && d_cu == reinterpret_cast<int32_t *>(p + used - need + align_up_sz((size_t)h.k * 4, 256)) &&
            cudaMemcpyAsync(d_cu, h.d_cu, ((size_t)h.k + 1) * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return TD_ECUDA;
        if (h.data_elems && cudaMemcpyAsync(d_dat, h.d_data, (size_t)h.data_elems * esz, cudaMemcpyHostToDevice, st) !=
            cudaSuccess) return TD_ECUDA;
        dev[i].d_indices = d_idx; dev[i].d_cu = ragged ? d_cu : nullptr; dev[i].d_data = d_dat;
    }
    return td_put_many(d, dev.data(), n_items, stream);
}

}  // extern "C"
