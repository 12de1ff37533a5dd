// td_get: readiness scan + compaction + claim (select), cu_seqlens / advantages (finalize),
// ragged gather.  Workflow steps 1 and 2 of "Distributed Transfer Dock Strategy": the worker
// state asks its controller which samples come next, then fetches the real data.
#pragma once

#include "td_device.cuh"

namespace td {

constexpr int kSelThreads = 256;            // one thread per group; a tile is 256 groups
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kFinThreads = 256;            // finalize: threads per request; kFinThreadsBig when a request is large
constexpr int kFinThreadsBig = 1024;
constexpr uint32_t kFinBigSamples = 1024;   // a request that may serve more samples than this gets the large block
constexpr uint32_t kFinGroupsKept = 1024;   // groups of a request whose numbers finalize keeps in shared memory
constexpr int kMaxJobs = 4096;              // (request, column) pairs one gather launch serves
// A request that wants the fused token stream has three more jobs behind its columns: the
// stream's prompt half, its response half, and the advantage twin.
constexpr uint32_t kSeqJobs = 3;

// Tile descriptor of the single-pass scan: [63:32] launch sequence number, [31:30] state,
// [29:0] count.  A descriptor whose sequence number is not the launch's is "not written yet",
// so scratch never has to be cleared between gets.
constexpr uint32_t kStateAggregate = 1, kStatePrefix = 2, kStateFailed = 3;
__host__ __device__ __forceinline__ unsigned long long desc_pack(uint32_t seq, uint32_t state, uint32_t count) {
    return ((unsigned long long)seq << 32) | ((unsigned long long)state << 30) | (count & 0x3fffffffu);
}
__device__ __forceinline__ uint32_t desc_seq(unsigned long long d) { return (uint32_t)(d >> 32); }
__device__ __forceinline__ uint32_t desc_state(unsigned long long d) { return (uint32_t)(d >> 30) & 3u; }
__device__ __forceinline__ uint32_t desc_count(unsigned long long d) { return (uint32_t)d & 0x3fffffffu; }

// Scratch of one (call, consumer): [0] ticket, [1] the gather's chunk counter, [2 .. 2+T) tile
// descriptors, then uint32[T] (padded to a multiple of 8 bytes) the exclusive rank each tile
// started from, then the candidate list int32[G]: the r-th ready group in index order, one's
// complement when the claim was lost to a concurrent get.
struct SelScratch {
    unsigned long long *ticket;
    unsigned long long *desc;
    uint32_t *excl;
    int32_t *cand;
};
// A tile is 256 groups per pass; a dock of more than kSelWideFrom groups gives every tile
// kSelWide passes (the tiles' tickets and descriptors are a serial chain: about 10 ns per tile,
// which outweighs the status words once there are thousands of tiles).
constexpr uint32_t kSelWide = 4, kSelWideFrom = 65536;
__host__ __device__ constexpr uint32_t sel_passes(uint32_t G) { return G > kSelWideFrom ? kSelWide : 1u; }
__host__ __device__ constexpr uint32_t sel_tiles(uint32_t G) {
    return (G + kSelThreads * sel_passes(G) - 1) / (kSelThreads * sel_passes(G));
}
__host__ __device__ constexpr size_t sel_excl_bytes(uint32_t G) { return (((size_t)sel_tiles(G) * 4) + 7) & ~size_t(7); }
__host__ __device__ constexpr size_t sel_scratch_bytes(uint32_t G) {
    return ((2 + (size_t)sel_tiles(G)) * 8 + sel_excl_bytes(G) + (size_t)G * 4 + 15) & ~size_t(15);
}
__host__ __device__ __forceinline__ SelScratch sel_scratch(void *p, uint32_t G) {
    SelScratch s;
    s.ticket = reinterpret_cast<unsigned long long *>(p);
    s.desc = s.ticket + 2;
    s.excl = reinterpret_cast<uint32_t *>(s.desc + sel_tiles(G));
    s.cand = reinterpret_cast<int32_t *>(reinterpret_cast<uint8_t *>(s.excl) + sel_excl_bytes(G));
    return s;
}

// One request of a call and the consumer slot it draws its groups from.  The kernels read a
// request's fields from global memory chunk after chunk: a size that is a whole number of
// 128-byte lines keeps every field of every request of a plan inside one 32-byte sector (with
// the struct at 656 bytes a drain of 128 requests took 2 us longer).
struct alignas(128) GetReq {
    td_get_out out;
    uint32_t consumer;
    uint32_t max_groups;      // floor(max_samples / N)
    uint32_t rank_base;       // first candidate rank this request may take
    uint32_t cslot;
    // Plans only: where, in a staging buffer that a call may bring along, a second copy of the
    // request's small outputs goes, so that a caller with host buffers fetches those of all
    // requests with one transfer.  Layout of the block: td_result, indices[m], cu_prompt[m+1],
    // cu_response[m+1], cu_seq[m+1], advantages[m], m = meta_samples.
    uint64_t meta_off;
    uint32_t meta_samples;
    // What the output buffers leave room for, worked out on the host when the request is set up
    // (the finalize kernel would otherwise walk the column pointers and capacities one dependent
    // load after the other): samples by the tightest scalar column, prompt / response tokens by the
    // tightest packed column of the class, rows by the tightest padded column; which classes
    // have a wanted ragged column at all.
    uint32_t want_classes;     // bit 1: a prompt-length column is wanted, bit 2: a response-length one
    uint64_t room_tok[3];
    uint64_t room_rows;
};
static_assert(sizeof(GetReq) == 768, "requests of a plan are read in whole 128-byte lines");
// Views into such a block.
struct MetaView {
    td_result *result;
    int32_t *indices, *cu_prompt, *cu_response, *cu_seq;
    float *advantages;
};
__host__ __device__ __forceinline__ size_t meta_bytes(uint32_t m) {
    return sizeof(td_result) + ((size_t)m * 2 + 3 * ((size_t)m + 1)) * 4;
}
__host__ __device__ __forceinline__ MetaView meta_view(uint8_t *p, uint32_t m) {
    MetaView v;
    v.result = reinterpret_cast<td_result *>(p);
    v.indices = reinterpret_cast<int32_t *>(p + sizeof(td_result));
    v.cu_prompt = v.indices + m;
    v.cu_response = v.cu_prompt + (m + 1);
    v.cu_seq = v.cu_response + (m + 1);
    v.advantages = reinterpret_cast<float *>(v.cu_seq + (m + 1));
    return v;
}
struct ConsumerSlot {
    uint32_t consumer;
    uint32_t max_groups;      // over all requests of the call that name this consumer
    void *scratch;
};
struct GetInline {            // a single get travels in the kernel parameters
    GetReq req;
    ConsumerSlot cs;
};

// The two halves of a tile's work, around whatever tells it how many ready groups come before
// it.  select_eval: thread tid tests one group per pass (all N status words carry the
// consumer's need bits, the group is not claimed) and the tile's ready groups are counted by
// warp ballots.  select_claim: the ready groups whose rank is below max_groups are claimed with
// one atomicOr per warp and pass and entered into the candidate list.
template <int kPasses>
struct TileState {
    bool ready[kPasses];
    uint32_t in_warp[kPasses];   // ready groups before this lane in its warp, per pass
    uint32_t before[kPasses];    // ready groups of the tile before this thread's warp and pass
    uint32_t g0;                 // group of pass 0
};
template <int kPasses>
__device__ __forceinline__ uint32_t select_eval(const DockView &dv, const uint32_t *claim, uint32_t need, uint32_t tile,
                                                uint32_t (*s_warp)[kSelWarps], TileState<kPasses> &ts) {
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // pass u of the tile covers groups [tile * kPasses + u] * 256 ...: thread tid tests one of them
    ts.g0 = tile * (kSelThreads * kPasses) + tid;
    // The claim word and the group's N status words are read with relaxed loads, all in flight
    // together (four words per load when N allows), and one fence behind them makes the set an
    // acquire: a status bit seen here was published after its payload, and the gather that
    // follows in this stream reads that payload.
    #pragma unroll
    for (int u = 0; u < kPasses; ++u) {
        const uint32_t g = ts.g0 + (uint32_t)u * kSelThreads;
        ts.ready[u] = false;
        if (g < dv.G) {
            const uint32_t cw = ld_relaxed_u32(&claim[g >> 5]);
            const uint32_t *st = dv.status + (size_t)g * dv.N;
            uint32_t all = need;
            if ((dv.N & 3u) == 0) {
                #pragma unroll 8
                for (uint32_t j = 0; j < dv.N; j += 4) {
                    const uint4 w = ld_relaxed_u32x4(st + j);
                    all &= w.x & w.y & w.z & w.w;
                }
            } else {
                #pragma unroll 4
                for (uint32_t j = 0; j < dv.N; ++j) all &= ld_relaxed_u32(st + j);
            }
            ts.ready[u] = !((cw >> (g & 31)) & 1u) && all == need;
        }
    }
    __threadfence();
    #pragma unroll
    for (int u = 0; u < kPasses; ++u) {
        const uint32_t ballot = __ballot_sync(kFullMask, ts.ready[u]);
        ts.in_warp[u] = __popc(ballot & ((1u << lane) - 1u));
        if (lane == 0) s_warp[u][warp] = __popc(ballot);
    }
    __syncthreads();
    uint32_t tile_count = 0;
    #pragma unroll
    for (int u = 0; u < kPasses; ++u) {
        ts.before[u] = tile_count;
        #pragma unroll
        for (int w = 0; w < kSelWarps; ++w) {
            const uint32_t v = s_warp[u][w];
            if (w < (int)warp) ts.before[u] += v;
            tile_count += v;
        }
    }
    return tile_count;
}
template <int kPasses>
__device__ __forceinline__ void select_claim(const DockView &dv, uint32_t *claim, const SelScratch &sc, uint32_t excl,
                                             uint32_t max_groups, const TileState<kPasses> &ts) {
    const uint32_t lane = threadIdx.x & 31;
    #pragma unroll
    for (int u = 0; u < kPasses; ++u) {
        const uint32_t g = ts.g0 + (uint32_t)u * kSelThreads;
        const uint32_t rank = excl + ts.before[u] + ts.in_warp[u];
        const bool cand = ts.ready[u] && rank < max_groups;
        const uint32_t mask = __ballot_sync(kFullMask, cand);
        uint32_t old = 0;
        if (lane == 0 && mask) old = atomicOr(&claim[g >> 5], mask);   // the warp's 32 groups share a word
        old = __shfl_sync(kFullMask, old, 0);
        if (cand) sc.cand[rank] = ((old >> lane) & 1u) ? ~(int32_t)g : (int32_t)g;
        const uint32_t lost = __popc(mask & old);
        if (lane == 0 && lost) atomicAdd(&dv.counters[CNT_CONFLICT], (unsigned long long)lost);
    }
}

// ---------------------------------------------------------------------------------------------
// Select.  grid = (tiles, consumer slots).  Thread g of a tile tests group g: all N status
// words carry the consumer's need bits and the group is not claimed.  Warp ballots and popc
// give the rank inside the tile, a decoupled look-back over the tile descriptors gives the
// rank before it, and the first max_groups ready groups are claimed with one atomicOr per
// warp.  Tiles take their number from a ticket, so a tile only ever waits for tiles that have
// already started; the wait is bounded all the same (dv.lookback_limit polls).  A tile that gives
// up marks its descriptor failed and claims nothing; the tiles ahead of it may already have
// claimed, which is why a tile records the rank it started from before it publishes its prefix:
// the finalize kernel, which serves nothing from a scan that did not come through, hands exactly
// those claims back.
// ---------------------------------------------------------------------------------------------
template <int kPasses>
__global__ void __launch_bounds__(kSelThreads)
get_select_kernel(const DockView dv, const __grid_constant__ GetInline one,
                  const ConsumerSlot *slots_dev, const uint32_t seq) {
    const ConsumerSlot *slots = slots_dev ? slots_dev : &one.cs;
    const ConsumerSlot cs = slots[blockIdx.y];
    const SelScratch sc = sel_scratch(cs.scratch, dv.G);
    const uint32_t c = cs.consumer;
    const uint32_t need = dv.need[c];
    uint32_t *claim = dv.claim + (size_t)c * dv.claim_words;
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ uint32_t s_tile, s_excl, s_failed;
    __shared__ uint32_t s_warp[kPasses][kSelWarps];
    griddep_launch_dependents();
    griddep_wait();                                    // status and claim words as the work before this call left them

    if (tid == 0) {
        // ticket word = seq << 32 | tiles started; sequence numbers only grow
        atomicMax(sc.ticket, (unsigned long long)seq << 32);
        const unsigned long long t = atomicAdd(sc.ticket, 1ull);
        s_tile = (uint32_t)(t & 0xffffffffu);
        // scratch shared with another launch in flight: refuse rather than index past the tiles
        s_failed = (uint32_t)(t >> 32) != seq || (uint32_t)(t & 0xffffffffu) >= gridDim.x;
    }
    __syncthreads();
    if (s_failed) {
        if (tid == 0) flag_error(dv, TD_ERR_LOOKBACK_TIMEOUT, CNT_TIMEOUT);
        return;
    }
    const uint32_t tile = s_tile;
    if (tile == dv.debug_skip_tile) return;            // test hook: this tile never shows up; its successors' waits run out
    TileState<kPasses> ts;
    const uint32_t tile_count = select_eval<kPasses>(dv, claim, need, tile, s_warp, ts);

    if (warp == 0) {
        uint32_t excl = 0;
        bool failed = s_failed;
        if (tile == 0) {
            if (lane == 0) {
                sc.excl[0] = 0;
                st_release_u64(&sc.desc[0], desc_pack(seq, kStatePrefix, tile_count));
            }
        } else {
            if (lane == 0) st_release_u64(&sc.desc[tile], desc_pack(seq, kStateAggregate, tile_count));
            // look back over windows of 32 predecessors
            int32_t look = (int32_t)tile - 1;
            bool done = false;
            while (!done && !failed) {
                const int32_t t = look - (int32_t)lane;
                unsigned long long d = 0;
                uint32_t state = kStatePrefix, count = 0;     // lanes before tile 0 contribute nothing
                if (t >= 0) {
                    uint32_t polls = 0;
                    do {
                        d = ld_acquire_u64(&sc.desc[t]);
                        if (desc_seq(d) == seq && desc_state(d) != 0) break;
                        __nanosleep(32);
                    } while (++polls < dv.lookback_limit);
                    if (desc_seq(d) != seq || desc_state(d) == 0) state = kStateFailed;
                    else { state = desc_state(d); count = desc_count(d); }
                }
                const uint32_t bad = __ballot_sync(kFullMask, state == kStateFailed);
                const uint32_t pre = __ballot_sync(kFullMask, state == kStatePrefix);
                // nearest predecessor that already knows its inclusive prefix
                const uint32_t first = pre ? (uint32_t)__ffs(pre) - 1u : 32u;
                const uint32_t upto = first < 32u ? first : 31u;
                if (bad & (upto == 31u ? kFullMask : ((2u << upto) - 1u))) { failed = true; break; }
                excl += __reduce_add_sync(kFullMask, lane <= upto ? count : 0u);
                if (first < 32u) done = true; else look -= 32;
            }
            if (lane == 0) {
                if (!failed) sc.excl[tile] = excl;     // ordered ahead of the descriptor by its release
                st_release_u64(&sc.desc[tile], failed ? desc_pack(seq, kStateFailed, 0)
                                                      : desc_pack(seq, kStatePrefix, excl + tile_count));
            }
        }
        if (lane == 0) { s_excl = excl; s_failed = failed; }
    }
    __syncthreads();
    if (s_failed) {
        if (tid == 0) flag_error(dv, TD_ERR_LOOKBACK_TIMEOUT, CNT_TIMEOUT);
        return;
    }
    select_claim<kPasses>(dv, claim, sc, s_excl, cs.max_groups, ts);
}

// ---------------------------------------------------------------------------------------------
// Finalize.  One CTA per request: compacts the groups it won into `indices`, builds
// cu_prompt / cu_response / cu_seq by block scans, cuts the batch before the first group that
// would not fit a supplied buffer (handing the cut groups back), sets the consumed bits,
// computes the group-normalised advantages and writes the result block.
// ---------------------------------------------------------------------------------------------
template <int kThreads>
__device__ __forceinline__ uint64_t block_scan_incl_2(uint64_t a, uint64_t b, uint64_t &out_b,
                                                      uint64_t *sh_a, uint64_t *sh_b,
                                                      uint64_t &tot_a, uint64_t &tot_b) {
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    #pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint64_t ta = __shfl_up_sync(kFullMask, a, d);
        const uint64_t tb = __shfl_up_sync(kFullMask, b, d);
        if ((int)lane >= d) { a += ta; b += tb; }
    }
    __syncthreads();                 // previous use of sh_* finished
    if (lane == 31) { sh_a[warp] = a; sh_b[warp] = b; }
    __syncthreads();
    uint64_t oa = 0, ob = 0; tot_a = 0; tot_b = 0;
    #pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
        if (w < (int)warp) { oa += sh_a[w]; ob += sh_b[w]; }
        tot_a += sh_a[w]; tot_b += sh_b[w];
    }
    out_b = b + ob;
    return a + oa;
}

// Output bytes of column k of a request that serves n_s samples with these token totals.
__device__ __forceinline__ uint64_t job_bytes_of(const DockView &dv, const GetReq &rq, uint32_t k,
                                                 uint64_t n_s, uint64_t prompt_tokens, uint64_t response_tokens) {
    const td_get_out &out = rq.out;
    if (k >= dv.ncol) {
        const uint32_t v = k - dv.ncol;
        if (v == 2) return out.seq_advantages ? (prompt_tokens + response_tokens) * 4u : 0;
        if (!out.seq) return 0;
        return (v == 0 ? prompt_tokens : response_tokens) * dv.col_esz[out.seq_prompt_col];
    }
    if (!((dv.outm[rq.consumer] >> k) & 1u) || out.col[k] == nullptr) return 0;
    const uint32_t cls = dv.col_cls[k], esz = dv.col_esz[k];
    if (cls == TD_SCALAR) return n_s * esz;
    if (out.mode == TD_PACKED) return (cls == TD_PROMPT ? prompt_tokens : response_tokens) * esz;
    return n_s * (uint64_t)(cls == TD_PROMPT ? out.pad_prompt_to : out.pad_response_to) * esz;
}

// What the gather needs to know about a (request, column) pair before it touches the request.
struct JobSize {
    uint64_t bytes;       // output bytes of the column (not padded)
    uint32_t rows;        // samples served
    uint32_t cost_rows;   // rows that are charged kRowCost in the chunked space: those of a packed ragged column
};

// An element of a scalar column costs a warp two dependent loads and a store, far more than its
// four bytes say: in the space the gather cuts into chunks it takes kScalarCost bytes, so that a
// chunk never holds more than a few hundred of them.
constexpr uint32_t kScalarCost = 64;
static_assert(kScalarCost % 16 == 0, "a job's extent stays a multiple of 16");
// Jobs are laid end to end in the chunked space on multiples of kJobUnit bytes, and the gather
// keeps their ends as 32-bit counts of units: 2^32 units are 256 GiB of extent per launch.
constexpr uint32_t kJobUnit = 64;
constexpr uint64_t kMaxLaunchExtent = (uint64_t)kJobUnit << 32;

// Extent of a job in the space the gather cuts into chunks (see kRowCost).
__device__ __forceinline__ uint32_t job_cost_rows(const DockView &dv, const GetReq &rq, uint32_t k,
                                                  uint64_t bytes, uint32_t n_s) {
    if (k >= dv.ncol) return (bytes != 0 && k - dv.ncol < 2u) ? n_s : 0u;      // the stream's halves are packed rows
    return (bytes != 0 && dv.col_cls[k] != TD_SCALAR && rq.out.mode == TD_PACKED) ? n_s : 0u;
}

// kFused: the dock has at most one (wide) tile of groups and every consumer of the call one
// request, so the request's CTA does the scan and the claim itself first (one launch less).
template <int kThreads, bool kFused>
__global__ void __launch_bounds__(kThreads)
get_finalize_kernel(const DockView dv, const __grid_constant__ GetInline one,
                    const GetReq *reqs_dev, const ConsumerSlot *slots_dev, const uint32_t seq,
                    unsigned long long *work_counter, JobSize *job_sizes, const uint32_t jobs_per_req,
                    uint8_t *meta_base) {
    const GetReq *reqs = reqs_dev ? reqs_dev : &one.req;
    const ConsumerSlot *slots = slots_dev ? slots_dev : &one.cs;
    const GetReq &rq = reqs[blockIdx.x];
    const td_get_out &out = rq.out;
    const ConsumerSlot cs = slots[rq.cslot];
    const SelScratch sc = sel_scratch(cs.scratch, dv.G);
    const uint32_t c = rq.consumer, N = dv.N;
    const uint32_t tid = threadIdx.x;
    const bool mirror = meta_base != nullptr;                    // the call brought a staging buffer along
    const MetaView mv = meta_view(meta_base + rq.meta_off, rq.meta_samples);
    __shared__ uint64_t sh_a[kThreads / 32], sh_b[kThreads / 32];
    __shared__ uint32_t s_first_over;
    // the groups served, for the first kFinGroupsKept of them: later steps take a sample's index
    // from here instead of reading the index list back from global memory
    __shared__ int32_t s_grp[kFinGroupsKept];
    griddep_launch_dependents();
    griddep_wait();                                    // the scan's candidate list is complete
    if (blockIdx.x == 0 && threadIdx.x == 0) *work_counter = 0;     // the gather hands out its chunks from zero

    uint32_t status = 0;
    uint32_t total = 0;
    int32_t g_first = -1;
    if constexpr (kFused) {
        static_assert(!kFused || kThreads == kSelThreads, "the fused scan is one tile of kSelThreads threads");
        __shared__ uint32_t s_warp[kSelWide][kSelWarps];
        uint32_t *claim = dv.claim + (size_t)c * dv.claim_words;
        TileState<(int)kSelWide> ts;
        const uint32_t tile_count = select_eval<(int)kSelWide>(dv, claim, dv.need[c], 0u, s_warp, ts);
        select_claim<(int)kSelWide>(dv, claim, sc, 0u, cs.max_groups, ts);
        __syncthreads();                                   // the consumer's candidate list is complete
        total = min(tile_count, cs.max_groups);
        if (tid < rq.max_groups && rq.rank_base + tid < dv.G) g_first = sc.cand[rq.rank_base + tid];
    } else {
        // how many groups were ready, from the last tile's inclusive prefix; the first candidates
        // are asked for in the same breath (which of them count is known once the prefix is here)
        const uint32_t tiles = sel_tiles(dv.G);
        const unsigned long long last = sc.desc[tiles - 1];
        if (tid < rq.max_groups && rq.rank_base + tid < dv.G) g_first = sc.cand[rq.rank_base + tid];
        // Every tile must have come through, not only the last one: a tile may give up on a slow
        // predecessor that its own successors still catch, and its ranks of the candidate list
        // are then never written.
        bool bad = false;
        for (uint32_t t = tid; t < tiles; t += kThreads) {
            const unsigned long long d = t == tiles - 1 ? last : sc.desc[t];
            bad |= desc_seq(d) != seq || desc_state(d) != kStatePrefix;
        }
        if (__syncthreads_or(bad)) {
            // Nothing is served from this scan.  The tiles that did come through have claimed
            // their groups (ranks [excl, inclusive prefix) below the consumer's limit, except the
            // ones lost to another get): the consumer's first request of the call gives them back.
            status |= TD_ERR_LOOKBACK_TIMEOUT;
            if (rq.rank_base == 0) {
                if (tid == 0) atomicAdd(&dv.counters[CNT_TIMEOUT], 1ull);      // once per consumer and call, whatever the tiles counted
                uint32_t *claim = dv.claim + (size_t)c * dv.claim_words;
                for (uint32_t t = tid; t < tiles; t += kThreads) {
                    const unsigned long long d = sc.desc[t];
                    if (desc_seq(d) != seq || desc_state(d) != kStatePrefix) continue;
                    const uint32_t r1 = min(desc_count(d), cs.max_groups);
                    for (uint32_t r = sc.excl[t]; r < r1; ++r) {
                        const int32_t g = sc.cand[r];
                        if (g >= 0) atomicAnd(&claim[(uint32_t)g >> 5], ~(1u << ((uint32_t)g & 31)));
                    }
                }
            }
        } else {
            total = min(desc_count(last), cs.max_groups);
        }
    }
    const uint32_t lo = rq.rank_base;
    const uint32_t hi = min(lo + rq.max_groups, total);
    const uint32_t ncand = hi > lo ? hi - lo : 0;

    // pass A: groups won, in order -> indices
    uint32_t n_grp = 0;
    for (uint32_t base = 0; base < ncand; base += kThreads) {
        const uint32_t r = base + tid;
        int32_t g = -1;
        if (r < ncand) g = base == 0 ? g_first : sc.cand[lo + r];
        uint64_t dummy_b, ta, tb;
        const uint64_t inc = block_scan_incl_2<kThreads>(g >= 0 ? 1u : 0u, 0, dummy_b, sh_a, sh_b, ta, tb);
        if (g >= 0) {
            const uint32_t p = n_grp + (uint32_t)inc - 1u;
            if (p < kFinGroupsKept) s_grp[p] = g;
            for (uint32_t j = 0; j < N; ++j) out.indices[(size_t)p * N + j] = g * (int32_t)N + (int32_t)j;
            if (mirror)
                for (uint32_t j = 0; j < N; ++j) mv.indices[(size_t)p * N + j] = g * (int32_t)N + (int32_t)j;
        }
        n_grp += (uint32_t)ta;
    }
    __syncthreads();
    uint32_t n_s = n_grp * N;
    // the groups' rewards are wanted last, behind the cu scans: ask for their lines now
    if ((dv.cflags[c] & TD_F_ADVANTAGE) && tid < n_grp && tid < kFinGroupsKept) {
        const float *r = reinterpret_cast<const float *>(dv.colbase[dv.reward_col]) + (size_t)s_grp[tid] * N;
        asm volatile("prefetch.global.L1 [%0];" ::"l"(r));
        if (N > 32u) asm volatile("prefetch.global.L1 [%0];" ::"l"(r + N - 1));
    }
    // A request of at most 32 groups has its groups' statistics worked out now, by the lanes of the
    // block's last warp, one group each, while the first warps are at the cu scans: the reward
    // loads and the double-precision sums then wait side by side with the length loads instead
    // of behind them.  (Groups that the fit test below cuts off were looked at in vain.)
    const bool adv_wanted = (dv.cflags[c] & TD_F_ADVANTAGE) && out.advantages;
    const bool adv_early = adv_wanted && n_grp <= 32u;
    __shared__ double s_mean[32], s_den[32];
    if (adv_early && tid >= (uint32_t)kThreads - 32u && tid - ((uint32_t)kThreads - 32u) < n_grp) {
        const uint32_t p = tid - ((uint32_t)kThreads - 32u);
        const float *r = reinterpret_cast<const float *>(dv.colbase[dv.reward_col]) + (size_t)s_grp[p] * N;
        double sum = 0.0;
        for (uint32_t j = 0; j < N; ++j) sum += (double)r[j];
        const double mean = sum / (double)N;
        double ss = 0.0;
        for (uint32_t j = 0; j < N; ++j) { const double d = (double)r[j] - mean; ss += d * d; }
        s_mean[p] = mean;
        s_den[p] = sqrt(ss / (double)N) + dv.eps;
    }
    const FastDiv div_N = make_fastdiv_dev(N);
    // sample at position i of the batch
    auto sample_at = [&](uint32_t i) -> int32_t {
        const uint32_t p = fast_div(i, div_N);
        return p < kFinGroupsKept ? s_grp[p] * (int32_t)N + (int32_t)(i - p * N) : out.indices[i];
    };

    // pass B: cu_seqlens and the fit test
    if (tid == 0) {
        s_first_over = 0xffffffffu;
        out.cu_prompt[0] = 0; out.cu_response[0] = 0;
        if (out.cu_seq) out.cu_seq[0] = 0;
        if (mirror) { mv.cu_prompt[0] = 0; mv.cu_response[0] = 0; mv.cu_seq[0] = 0; }
    }
    // tightest room per length class over the wanted columns (set up on the host)
    const uint64_t room_tok[3] = {rq.room_tok[0], rq.room_tok[1], rq.room_tok[2]};
    const uint64_t room_rows = rq.room_rows;
    const uint64_t room_seq = (out.seq || out.seq_advantages) ? out.seq_capacity_elems : ~0ull;
    const bool padded = out.mode == TD_PADDED;
    const bool want_p = (rq.want_classes >> TD_PROMPT) & 1u, want_r = (rq.want_classes >> TD_RESPONSE) & 1u;
    uint64_t carry_p = 0, carry_r = 0;
    for (uint32_t base = 0; base < n_s; base += kThreads) {
        const uint32_t i = base + tid;
        uint64_t lp = 0, lr = 0;
        if (i < n_s) {
            const int32_t s = sample_at(i);
            const int32_t a = dv.len[TD_PROMPT][s], b = dv.len[TD_RESPONSE][s];
            lp = a > 0 ? (uint64_t)a : 0; lr = b > 0 ? (uint64_t)b : 0;
        }
        uint64_t ir, tp, tr;
        const uint64_t ip = block_scan_incl_2<kThreads>(lp, lr, ir, sh_a, sh_b, tp, tr);
        if (i < n_s) {
            const uint64_t cp = carry_p + ip, cr = carry_r + ir;
            out.cu_prompt[i + 1] = (int32_t)cp;
            out.cu_response[i + 1] = (int32_t)cr;
            if (out.cu_seq) out.cu_seq[i + 1] = (int32_t)(cp + cr);
            if (mirror) {
                mv.cu_prompt[i + 1] = (int32_t)cp; mv.cu_response[i + 1] = (int32_t)cr;
                mv.cu_seq[i + 1] = (int32_t)(cp + cr);
            }
            bool over = (uint64_t)(i + 1) > room_tok[0];
            if (!padded) over |= cp > room_tok[TD_PROMPT] || cr > room_tok[TD_RESPONSE];
            else over |= (uint64_t)(i + 1) > room_rows || (want_p && lp > out.pad_prompt_to) ||
                         (want_r && lr > out.pad_response_to);
            over |= cp + cr > room_seq;
            if (over) atomicMin(&s_first_over, i);
        }
        carry_p += tp; carry_r += tr;
    }
    __syncthreads();
    uint64_t tot_p = carry_p, tot_r = carry_r;         // the batch's token totals
    if (s_first_over != 0xffffffffu) {
        const uint32_t keep = s_first_over / N;
        #pragma unroll 1
        for (uint32_t p = keep + tid; p < n_grp; p += kThreads) {
            const uint32_t g = (uint32_t)out.indices[(size_t)p * N] / N;
            atomicAnd(&dv.claim[(size_t)c * dv.claim_words + (g >> 5)], ~(1u << (g & 31)));
        }
        n_grp = keep; n_s = keep * N;
        status |= TD_ERR_OUT_TRUNCATED;
        if (tid == 0) flag_error(dv, TD_ERR_OUT_TRUNCATED, CNT_TRUNC);
        tot_p = (uint64_t)(int64_t)out.cu_prompt[n_s];            // the cut batch ends here
        tot_r = (uint64_t)(int64_t)out.cu_response[n_s];
    }
    // consumed bits
    uint32_t *consumed = dv.consumed + (size_t)c * dv.consumed_words;
    for (uint32_t i = tid; i < n_s; i += kThreads) {
        const uint32_t s = (uint32_t)sample_at(i);
        atomicOr(&consumed[s >> 5], 1u << (s & 31));
    }
    // group-normalised advantage in double: one thread per sample from the statistics taken
    // above, or (a large request) one thread per group
    if (adv_early) {
        const float *rew = reinterpret_cast<const float *>(dv.colbase[dv.reward_col]);
        for (uint32_t i = tid; i < n_s; i += kThreads) {
            const uint32_t p = fast_div(i, div_N);
            const float adv = (float)(((double)rew[sample_at(i)] - s_mean[p]) / s_den[p]);
            out.advantages[i] = adv;
            if (mirror) mv.advantages[i] = adv;
        }
    } else if (adv_wanted) {
        const float *rew = reinterpret_cast<const float *>(dv.colbase[dv.reward_col]);
        for (uint32_t p = tid; p < n_grp; p += kThreads) {
            const float *r = rew + (p < kFinGroupsKept ? s_grp[p] * (int32_t)N : out.indices[(size_t)p * N]);   // a group's samples are consecutive
            double sum = 0.0;
            for (uint32_t j = 0; j < N; ++j) sum += (double)r[j];
            const double mean = sum / (double)N;
            double ss = 0.0;
            for (uint32_t j = 0; j < N; ++j) { const double d = (double)r[j] - mean; ss += d * d; }
            const double sd = sqrt(ss / (double)N);
            for (uint32_t j = 0; j < N; ++j) {
                const float adv = (float)(((double)r[j] - mean) / (sd + dv.eps));
                out.advantages[(size_t)p * N + j] = adv;
                if (mirror) mv.advantages[(size_t)p * N + j] = adv;
            }
        }
    }
    __syncthreads();
    if (tid == 0) {
        td_result r;
        r.n_samples = n_s; r.n_groups = n_grp;
        r.prompt_tokens = tot_p;
        r.response_tokens = tot_r;
        r.status = status; r.reserved = 0;
        *out.result = r;
        if (mirror) *mv.result = r;
        if (status & TD_ERR_LOOKBACK_TIMEOUT) atomicOr(dv.errword, TD_ERR_LOOKBACK_TIMEOUT);
        atomicAdd(&dv.counters[CNT_GOT_SAMPLES + c], (unsigned long long)n_s);
        atomicAdd(&dv.counters[CNT_GOT_TOKENS + c], (unsigned long long)(r.prompt_tokens + r.response_tokens));
    }
    // the gather's job table: this request's output bytes per column and its row count
    if (job_sizes && tid < jobs_per_req) {
        JobSize js;
        js.bytes = job_bytes_of(dv, rq, tid, n_s, tot_p, tot_r);
        js.rows = n_s;
        js.cost_rows = job_cost_rows(dv, rq, tid, js.bytes, n_s);
        job_sizes[(size_t)blockIdx.x * jobs_per_req + tid] = js;
    }
}

// ---------------------------------------------------------------------------------------------
// Gather.  Persistent grid.  Every (request, column) pair is a job; the jobs' extents (output
// bytes, plus kRowCost per row of a packed ragged column) are laid end to end and cut into
// chunks that warps take one after the other, so the work is balanced whatever the mix of
// requests and row lengths (see "Chunked ragged copy" in td_device.cuh).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ JobSize job_size(const DockView &dv, const GetReq &rq, uint32_t k) {
    const td_result *res = rq.out.result;
    JobSize js;
    js.rows = res->n_samples;
    js.bytes = job_bytes_of(dv, rq, k, js.rows, res->prompt_tokens, res->response_tokens);
    js.cost_rows = job_cost_rows(dv, rq, k, js.bytes, js.rows);
    return js;
}

// The advantage twin of the fused stream, bytes [b0, b1) of it: sample i's prompt tokens get 0,
// its response tokens its advantage.  Lane l looks row r0 + l up, the warp fills row by row.
__device__ __noinline__ void warp_fill_seq_advantages(const td_get_out &out, uint32_t n_s, uint64_t b0,
                                                      uint64_t b1, uint32_t lane) {
    if (b1 <= b0) return;
    const int32_t *cs = out.cu_seq, *cp = out.cu_prompt;
    uint8_t *dst = reinterpret_cast<uint8_t *>(out.seq_advantages);
    uint32_t r0 = warp_find_row(cs, n_s, (int64_t)b0, 4u, 0u, lane);
    for (;;) {
        const uint32_t i = r0 + lane;
        uint64_t lo = 0, mid = 0, hi = 0;
        uint32_t bits = 0;
        bool in = false;
        if (i < n_s) {
            lo = (uint64_t)__ldg(cs + i) * 4u;
            in = lo < b1;
            if (in) {
                hi = (uint64_t)__ldg(cs + i + 1) * 4u;
                mid = lo + (uint64_t)(__ldg(cp + i + 1) - __ldg(cp + i)) * 4u;
                bits = __float_as_uint(out.advantages[i]);
            }
        }
        const uint32_t inside = __ballot_sync(kFullMask, in);            // a prefix of the lanes
        const uint32_t n_rows = (uint32_t)__popc(inside);
        for (uint32_t r = 0; r < n_rows; ++r) {
            const uint64_t rlo = shfl_u64(lo, r), rmid = shfl_u64(mid, r), rhi = shfl_u64(hi, r);
            const uint32_t a = __shfl_sync(kFullMask, bits, r);
            const uint64_t z0 = max(rlo, b0), z1 = min(rmid, b1);
            if (z1 > z0) warp_fill(dst + z0, z1 - z0, 0u, 4u, lane);
            const uint64_t a0 = max(rmid, b0), a1 = min(rhi, b1);
            if (a1 > a0) warp_fill(dst + a0, a1 - a0, a, 4u, lane);
        }
        if (n_rows < 32u) break;
        r0 += 32u;
    }
}

__global__ void __launch_bounds__(kCopyThreads, kCopyBlocksPerSM)
get_gather_kernel(const DockView dv, const __grid_constant__ GetInline one,
                  const GetReq *reqs_dev, const uint32_t n_req, unsigned long long *work_counter,
                  const JobSize *job_sizes, const uint32_t jpr, const FastDiv div_jpr,
                  const ConsumerSlot *slots_dev, const uint32_t n_slots) {
    const GetReq *reqs = reqs_dev ? reqs_dev : &one.req;
    extern __shared__ __align__(128) uint8_t gather_smem[];
    uint64_t *s_wsum = reinterpret_cast<uint64_t *>(gather_smem + (size_t)kCopyWarps * kPipeSmemPerWarp);
    // [n_req * jpr] inclusive prefix of the jobs' extents in units of kJobUnit bytes, each job
    // rounded up to a whole unit (four bytes per job: a plan of thousands of jobs still leaves
    // room for two CTAs per SM).  With this and the rows served per request in shared memory, a
    // chunk's warp needs neither the result block nor the last cu entry; that a job's last
    // chunk reaches a few bytes past its true end does no harm, rows and elements bound it.
    uint32_t *job_end = reinterpret_cast<uint32_t *>(s_wsum + kCopyWarps);
    uint32_t *req_rows = job_end + n_req * jpr;                                       // [n_req]
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    WarpPipe pipe;
    pipe.init(gather_smem + (size_t)warp * kPipeSmemPerWarp, lane, dv.spin_limit);
    griddep_wait();                                    // indices, cu_seqlens and result blocks are complete
    // The scan and the finalize kernel are done with the scan scratch: leave its ticket and tile
    // descriptors empty for the next call, so that a call which comes with the same launch
    // sequence number again (a CUDA graph replayed) does not meet its own earlier descriptors.
    if (blockIdx.x == 0) {
        const ConsumerSlot *slots = slots_dev ? slots_dev : &one.cs;
        const uint32_t tiles = sel_tiles(dv.G);
        for (uint32_t i = threadIdx.x; i < n_slots * (tiles + 1u); i += kCopyThreads) {
            const uint32_t sl = i / (tiles + 1u), t = i - sl * (tiles + 1u);
            const SelScratch sc = sel_scratch(slots[sl].scratch, dv.G);
            if (t == tiles) *sc.ticket = 0; else sc.desc[t] = 0;
        }
    }
    const uint32_t ncol = dv.ncol;                     // jpr = ncol, or ncol + kSeqJobs when a request wants the stream
    const uint32_t njobs = n_req * jpr;

    // job table: sizes first (strided over the threads, so the dependent loads behind each
    // size - request, result block - are all in flight together), then one block scan in which
    // each thread owns a contiguous run
    {
        const uint32_t per = (njobs + kCopyThreads - 1) / kCopyThreads;
        #pragma unroll 4
        for (uint32_t i = 0; i < per; ++i) {
            const uint32_t j = i * kCopyThreads + tid;
            if (j < njobs) {
                JobSize js;
                if (job_sizes) {
                    js = job_sizes[j];                         // written by the finalize kernel
                } else {
                    const uint32_t q = fast_div(j, div_jpr);
                    js = job_size(dv, reqs[q], j - q * jpr);
                }
                const uint32_t q = fast_div(j, div_jpr);
                const uint32_t k = j - q * jpr;
                const bool scalar = k < ncol && dv.col_cls[k] == TD_SCALAR;
                const uint64_t extent = scalar ? (js.bytes ? (uint64_t)js.rows * kScalarCost : 0)
                                               : js.bytes + (uint64_t)js.cost_rows * kRowCost;
                job_end[j] = (uint32_t)((extent + (kJobUnit - 1)) / kJobUnit);
                if (k == 0) req_rows[q] = js.rows;
            }
        }
        __syncthreads();
        const uint32_t j0 = min(tid * per, njobs), j1 = min(j0 + per, njobs);
        uint64_t local = 0;
        for (uint32_t j = j0; j < j1; ++j) local += job_end[j];
        uint64_t inc = local;
        #pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint64_t t = shfl_up_u64(inc, d);
            if ((int)lane >= d) inc += t;
        }
        if (lane == 31) s_wsum[warp] = inc;
        __syncthreads();
        uint64_t run = inc - local;
        for (uint32_t w = 0; w < warp; ++w) run += s_wsum[w];
        for (uint32_t j = j0; j < j1; ++j) {               // the host has checked that the total fits 32 bits of units
            run += job_end[j];
            job_end[j] = (uint32_t)run;
        }
        __syncthreads();
    }
    const uint64_t total_all = njobs ? (uint64_t)job_end[njobs - 1] * kJobUnit : 0;
    const uint64_t n_warps = (uint64_t)gridDim.x * kCopyWarps;
    // A warp starts on the chunk of its own number; the chunks after the first n_warps are
    // handed out by a counter in scratch memory (zeroed by the finalize kernel): equal bytes are
    // not equal time when one chunk holds a few long rows and another many short ones.
    const ChunkPlan plan = plan_chunks_dynamic(total_all, n_warps);
    unsigned long long ch = (uint64_t)blockIdx.x * kCopyWarps + warp;

    while (ch < plan.n_chunks) {
        unsigned long long next = 0;
        if (lane == 0) next = n_warps + atomicAdd(work_counter, 1ull);   // in flight while this chunk is copied
        uint64_t g0 = ch * plan.chunk_bytes;
        const uint64_t g1 = min(g0 + plan.chunk_bytes, total_all);
        // first job that reaches beyond g0
        uint32_t j = 0;
        { uint32_t jhi = njobs - 1; while (j < jhi) { const uint32_t m = (j + jhi) >> 1; if ((uint64_t)job_end[m] * kJobUnit > g0) jhi = m; else j = m + 1; } }
        for (; g0 < g1; ++j) {
            const uint64_t start = j ? (uint64_t)job_end[j - 1] * kJobUnit : 0;
            const uint64_t end = (uint64_t)job_end[j] * kJobUnit;
            const uint64_t b0 = g0 - start;
            g0 = min(g1, end);
            if (end == start) continue;               // empty job
            const uint32_t q = fast_div(j, div_jpr);
            uint32_t k = j - q * jpr;
            const GetReq &rq = reqs[q];
            const td_get_out &out = rq.out;
            const uint32_t n_s = req_rows[q];
            const uint64_t b1_raw = g0 - start;          // end of this warp's part of the job (it may lie in the job's padding)
            uint8_t *dst0;
            const int32_t *seq_cu = nullptr;             // set for the two halves of the fused stream
            bool seq_tail = false;
            if (k >= ncol) {
                const uint32_t v = k - ncol;
                if (v == 2) {
                    warp_fill_seq_advantages(out, n_s, b0, b1_raw, lane);
                    continue;
                }
                k = v == 0 ? out.seq_prompt_col : out.seq_response_col;
                seq_cu = out.cu_seq; seq_tail = v == 1;
                dst0 = reinterpret_cast<uint8_t *>(out.seq);
            } else {
                dst0 = reinterpret_cast<uint8_t *>(out.col[k]);
            }
            const uint32_t cls = dv.col_cls[k], esz = dv.col_esz[k];
            uint8_t *base = dv.colbase[k];
            const int32_t *indices = out.indices;

            if (cls == TD_SCALAR) {
                // element e belongs to the chunk that holds byte e * kScalarCost of the job; four
                // elements per lane are looked up side by side
                const uint32_t e0 = (uint32_t)((b0 + kScalarCost - 1) / kScalarCost);
                const uint32_t e1 = (uint32_t)min((b1_raw + kScalarCost - 1) / kScalarCost, (uint64_t)n_s);
                for (uint32_t e = e0 + lane; e < e1; e += 128) {
                    int32_t s[4];
                    uint32_t v[4];
                    #pragma unroll
                    for (int u = 0; u < 4; ++u) s[u] = e + 32u * u < e1 ? __ldg(indices + e + 32u * u) : -1;
                    #pragma unroll
                    for (int u = 0; u < 4; ++u)
                        v[u] = s[u] < 0 ? 0u : esz == 4 ? reinterpret_cast<const uint32_t *>(base)[s[u]]
                                                        : (uint32_t)reinterpret_cast<const uint16_t *>(base)[s[u]];
                    #pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (s[u] >= 0) {
                            if (esz == 4) reinterpret_cast<uint32_t *>(dst0)[e + 32u * u] = v[u];
                            else reinterpret_cast<uint16_t *>(dst0)[e + 32u * u] = (uint16_t)v[u];
                        }
                }
                continue;
            }
            const uint64_t cap = dv.cap[cls];
            const uint8_t *src_lo = base, *src_hi = base + (uint64_t)dv.S * cap * esz;
            const long long *offt = dv.off[cls];
            auto row_src = [&](uint32_t i) -> uint8_t * {
                const uint32_t s = (uint32_t)__ldg(indices + i);
                const long long off = offt[s];
                return off >= 0 ? base + ((uint64_t)shard_of(dv, s) * cap + (uint64_t)off) * esz : nullptr;
            };
            if (out.mode == TD_PACKED || seq_cu) {
                const int32_t *cu = cls == TD_PROMPT ? out.cu_prompt : out.cu_response;
                const uint64_t b1 = b1_raw;
                warp_copy_chunk<true, false>(cu, n_s, b0, b1, dst0, esz, lane, src_lo, src_hi, pipe, indices,
                                             [&](uint32_t i, int64_t, int64_t, int32_t &) -> uint8_t * { return row_src(i); },
                                             seq_cu, seq_tail);
            } else {
                // fixed-width rows: payload part, then the pad pattern up to the row's end; a
                // prompt row asked for left-padded has the pad pattern first and ends at its width
                const uint32_t W = cls == TD_PROMPT ? out.pad_prompt_to : out.pad_response_to;
                const uint64_t row_bytes = (uint64_t)W * esz;
                const uint64_t b1 = min(b1_raw, (uint64_t)n_s * row_bytes);
                const bool left = cls == TD_PROMPT && (out.flags & TD_OUT_LEFT_PAD_PROMPT);
                const int32_t *lent = dv.len[cls];
                for (uint64_t r0 = b0 / row_bytes; r0 < n_s && r0 * row_bytes < b1; r0 += 32) {
                    const uint64_t i = r0 + lane;
                    uint64_t valid = 0;
                    uint8_t *src = nullptr;
                    if (i < n_s && i * row_bytes < b1) {
                        const int32_t l = lent[(uint32_t)__ldg(indices + i)];
                        valid = (uint64_t)(l > 0 ? l : 0) * esz;
                        src = row_src((uint32_t)i);
                    }
                    for (uint32_t r = 0; r < 32; ++r) {
                        const uint64_t rlo = (r0 + r) * row_bytes;
                        if (r0 + r >= n_s || rlo >= b1) break;
                        // the row's payload lies at [v0, v1) of the job, this warp's part of the row is [lo, hi)
                        const uint64_t v_bytes = shfl_u64(valid, r);
                        const uint64_t v0 = left ? rlo + row_bytes - v_bytes : rlo, v1 = v0 + v_bytes;
                        uint8_t *o = reinterpret_cast<uint8_t *>(shfl_u64(reinterpret_cast<uint64_t>(src), r));
                        const uint64_t lo = max(rlo, b0), hi = min(rlo + row_bytes, b1);
                        const uint64_t p0 = max(lo, v0), p1 = min(hi, v1);
                        if (p1 > p0 && o)
                            pipe.push<false>(dst0 + p0, o + (p0 - v0), (uint32_t)(p1 - p0), lane, src_lo, src_hi);
                        if (left) {
                            const uint64_t fhi = min(hi, v0);
                            if (fhi > lo) warp_fill(dst0 + lo, fhi - lo, dv.col_pad[k], esz, lane);
                        } else {
                            const uint64_t flo = max(lo, v1);
                            if (hi > flo) warp_fill(dst0 + flo, hi - flo, dv.col_pad[k], esz, lane);
                        }
                    }
                }
            }
        }
        ch = shfl_u64(next, 0);
    }
    if (pipe.finish(lane) && lane == 0) flag_error(dv, TD_ERR_COPY_TIMEOUT, CNT_TIMEOUT);
}

// Reset: every table, bitmap and counter back to the empty state; payload untouched.
__global__ void __launch_bounds__(256)
reset_kernel(const DockView dv) {
    griddep_launch_dependents();                       // the first kernel of the next call may set itself up meanwhile
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t stride = gridDim.x * blockDim.x;
    for (uint32_t s = t; s < dv.n; s += stride) {
        dv.status[s] = 0;
        dv.len[1][s] = -1; dv.len[2][s] = -1;
        dv.off[1][s] = -1; dv.off[2][s] = -1;
    }
    for (uint32_t i = t; i < dv.S; i += stride) { dv.cursor[1][i] = 0; dv.cursor[2][i] = 0; }
    for (uint32_t i = t; i < dv.ncons * dv.claim_words; i += stride) dv.claim[i] = 0;
    for (uint32_t i = t; i < dv.ncons * dv.consumed_words; i += stride) dv.consumed[i] = 0;
    for (uint64_t i = t; i < (uint64_t)dv.ncol * dv.n; i += stride) dv.progress[i] = 0;
    for (uint32_t i = t; i < CNT_TOTAL; i += stride) dv.counters[i] = 0;
    if (t == 0) *dv.errword = 0;
}

}  // namespace td
