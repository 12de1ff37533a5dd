// Device-side view of a dock and the warp-level ragged copy shared by put and get.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/td.h"

namespace td {

constexpr int kMaxColumns = 32;
constexpr int kPutCounterSlots = 64;         // streams that can put into a dock with chunks handed out by a counter
constexpr uint32_t kRowAlign = 8;            // rows start on multiples of 8 elements (>= 16 bytes)
constexpr uint32_t kFullMask = 0xffffffffu;
// Internal bit of the dock's error word, never reported: a put since the last reset came with a
// cu array that is not a non-decreasing sequence inside [0, data_elems].  Row positions in such
// an array cannot be searched, so the scatter then takes its rows one by one.
constexpr uint32_t kErrIrregularCu = 1u << 31;

// counters[] slots (uint64 each)
enum : int {
    CNT_PUT_ACCEPTED = 0,    // + column
    CNT_GOT_SAMPLES = 32,    // + consumer
    CNT_GOT_TOKENS = 64,     // + consumer
    CNT_OOB = 96, CNT_DUP, CNT_MISMATCH, CNT_FULL, CNT_TRUNC, CNT_BADLEN, CNT_CONFLICT, CNT_TIMEOUT,
    CNT_TOTAL = 112
};

// Division by a run-time constant d through a multiply and a shift, exact for n < 2^31:
// n / d = (umulhi(n, mul) + n) >> shr with shr = ceil(log2 d), mul = floor(2^32 (2^shr - d) / d) + 1
// (mul = 0 when d is a power of two).
struct FastDiv {
    uint32_t mul, shr;
};
static inline FastDiv make_fastdiv(uint32_t d) {
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    const uint64_t m = (1ull << l) == d ? 0 : ((1ull << 32) * ((1ull << l) - d)) / d + 1;
    return FastDiv{(uint32_t)m, l};
}
__device__ __forceinline__ FastDiv make_fastdiv_dev(uint32_t d) {          // the same constants, computed on the device
    const uint32_t l = d > 1u ? 32u - (uint32_t)__clz(d - 1u) : 0u;
    const unsigned long long m = (1ull << l) == d ? 0ull : ((1ull << 32) * ((1ull << l) - d)) / d + 1ull;
    return FastDiv{(uint32_t)m, l};
}
__device__ __forceinline__ uint32_t fast_div(uint32_t n, FastDiv f) {
    return (__umulhi(n, f.mul) + n) >> f.shr;
}

// Everything a kernel needs to know about a dock; passed by value (constant bank).
struct DockView {
    uint32_t G, N, S, n;
    uint32_t ncol, ncons;
    uint32_t prompts_per_shard;
    uint32_t reward_col;
    FastDiv  div_shard;                     // by samples per shard = N * prompts_per_shard
    uint32_t claim_words, consumed_words;   // words per consumer
    uint32_t spin_limit;                    // polls before a wait on a staged copy gives up
    uint32_t lookback_limit;                // polls before a scan tile gives up waiting for a tile ahead of it
    uint32_t debug_skip_tile;               // test hook: the scan tile of this number withholds its descriptor (none: ~0u)
    uint32_t pad0;
    double   eps;
    uint64_t cap[3];                        // elements per shard, by length class
    uint32_t *status;                       // [n]
    int32_t  *len[3];                       // [n], -1 = unset           (index 1, 2)
    long long *off[3];                      // [n], -1 = unset
    unsigned long long *cursor[3];          // [S]
    uint32_t *claim;                        // [ncons][claim_words]
    uint32_t *consumed;                     // [ncons][consumed_words]
    uint32_t *errword;
    unsigned long long *counters;           // [CNT_TOTAL]
    unsigned long long *put_counters;       // [kPutCounterSlots] chunk counters of the scatter kernel, one per stream in use
    unsigned long long *put_ready;          // [kPutCounterSlots][4] per stream that puts: "inputs complete" word, entries allocated so far per length class (see PutBatch)
    uint32_t *progress;                     // [ncol][n] elements of a row written so far by the put that stores it
    uint8_t  *colbase[kMaxColumns];         // arena (S * cap * esz) or scalar store (n * esz)
    uint32_t need[kMaxColumns];             // per consumer
    uint32_t outm[kMaxColumns];
    uint32_t cflags[kMaxColumns];
    uint32_t col_pad[kMaxColumns];
    uint8_t  col_esz[kMaxColumns];
    uint8_t  col_cls[kMaxColumns];
};

// Warehouses hold contiguous blocks of whole prompts: shard(s) = (s / N) / (G / S).
__device__ __forceinline__ uint32_t shard_of(const DockView &dv, uint32_t s) {
    return fast_div(s, dv.div_shard);
}

__device__ __forceinline__ uint64_t align_row(uint64_t elems) {
    return (elems + (kRowAlign - 1)) & ~uint64_t(kRowAlign - 1);
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint4 ld_relaxed_u32x4(const uint32_t *p) {      // p is 16-byte aligned
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long *p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Programmatic dependent launch: the kernels of one call are chained so that the next one is
// launched, and runs its prologue, while the previous one is still finishing.  A kernel calls
// griddep_wait() before it touches anything the kernel before it in the stream wrote (the wait
// returns when that kernel has completed and its writes are visible; without the launch
// attribute it returns at once), and griddep_launch_dependents() as soon as the next kernel
// may be brought on.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void flag_error(const DockView &dv, uint32_t bit, int counter, uint32_t count = 1) {
    atomicOr(dv.errword, bit);
    atomicAdd(&dv.counters[counter], (unsigned long long)count);
}

// --------------------------------------------------------------------------------------------
// Warp-cooperative copy of n bytes from src to dst.  Both addresses and n are multiples of the
// element size (2 or 4 bytes); nothing else is assumed.  Two forms.  warp_copy is the plain one,
// word by word (half words when anything is odd), reading exactly the bytes it copies: it
// serves pieces too short to stage, pieces at the edge of a caller's buffer and the path after
// a failed wait, and is as small as it can be, because the instruction footprint of the copy
// kernels showed up in their speed.  warp_copy_from_shared is the one the data goes through:
// the source is a stage in shared memory, given as a shared-window address; stores are
// 16-byte vectors aligned on dst, each fed by four ld.shared.u32 (eight ld.shared.u16 when
// the two sides differ by an odd number of half words) at whatever phase the source has;
// head and tail move half words.
// --------------------------------------------------------------------------------------------
__device__ __noinline__ void warp_copy(uint8_t *dst, const uint8_t *src, uint32_t n, uint32_t lane) {
    if (((reinterpret_cast<uintptr_t>(dst) | reinterpret_cast<uintptr_t>(src) | n) & 3u) == 0) {
        for (uint32_t i = lane; i < (n >> 2); i += 32)
            reinterpret_cast<uint32_t *>(dst)[i] = reinterpret_cast<const uint32_t *>(src)[i];
    } else {
        for (uint32_t i = lane; i < (n >> 1); i += 32)
            reinterpret_cast<uint16_t *>(dst)[i] = reinterpret_cast<const uint16_t *>(src)[i];
    }
}

__device__ __forceinline__ uint32_t lds_u32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t a) {
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint4 lds_4x32(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.u32 %0, [%4];\n\tld.shared.u32 %1, [%4+4];\n\tld.shared.u32 %2, [%4+8];\n\tld.shared.u32 %3, [%4+12];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t smem_u32(const void *p);
__device__ __forceinline__ void warp_copy_from_shared(uint8_t *dst, uint32_t src, uint32_t n, uint32_t lane) {
    uint32_t head = (16u - (uint32_t)(reinterpret_cast<uintptr_t>(dst) & 15u)) & 15u;
    if (head > n) head = n;
    if (lane < (head >> 1)) reinterpret_cast<uint16_t *>(dst)[lane] = (uint16_t)lds_u16(src + 2u * lane);
    dst += head; src += head; n -= head;
    const uint32_t nvec = n >> 4;
    uint4 *D = reinterpret_cast<uint4 *>(dst);
    if ((src & 3u) == 0) {
        #pragma unroll 1                       // unrolled versions were measured slower
        for (uint32_t v = lane; v < nvec; v += 32) __stcs(D + v, lds_4x32(src + 16u * v));
    } else {
        #pragma unroll 1
        for (uint32_t v = lane; v < nvec; v += 32) {
            const uint32_t p = src + 16u * v;
            __stcs(D + v, make_uint4(lds_u16(p) | (lds_u16(p + 2) << 16), lds_u16(p + 4) | (lds_u16(p + 6) << 16),
                                     lds_u16(p + 8) | (lds_u16(p + 10) << 16), lds_u16(p + 12) | (lds_u16(p + 14) << 16)));
        }
    }
    const uint32_t tail = n & 15u;
    if (lane < (tail >> 1))
        reinterpret_cast<uint16_t *>(dst + (nvec << 4))[lane] = (uint16_t)lds_u16(src + (nvec << 4) + 2u * lane);
}

// Warp-cooperative fill of nbytes at dst (element aligned) with the element pattern `bits`.
__device__ __forceinline__ void warp_fill(uint8_t *dst, uint64_t nbytes, uint32_t bits, uint32_t esz,
                                          uint32_t lane) {
    if (nbytes == 0) return;
    const uint32_t word = esz == 4 ? bits : ((bits & 0xffffu) | (bits << 16));
    uint32_t head = (16u - (uint32_t)(reinterpret_cast<uintptr_t>(dst) & 15u)) & 15u;
    if (head > nbytes) head = (uint32_t)nbytes;
    if (head) {
        if (lane < head / esz) {
            if (esz == 4) reinterpret_cast<uint32_t *>(dst)[lane] = bits;
            else reinterpret_cast<uint16_t *>(dst)[lane] = (uint16_t)bits;
        }
        dst += head; nbytes -= head;
    }
    const uint64_t nvec = nbytes >> 4;
    uint4 *D = reinterpret_cast<uint4 *>(dst);
    const uint4 val = make_uint4(word, word, word, word);
    for (uint64_t v = lane; v < nvec; v += 32) __stcs(D + v, val);
    const uint32_t tail = (uint32_t)(nbytes & 15u);
    if (tail && lane < tail / esz) {
        uint8_t *t = dst + 16ull * nvec;
        if (esz == 4) reinterpret_cast<uint32_t *>(t)[lane] = bits;
        else reinterpret_cast<uint16_t *>(t)[lane] = (uint16_t)bits;
    }
}

// --------------------------------------------------------------------------------------------
// Chunked ragged copy.  The packed side of a ragged copy (the source of a put, the destination
// of a packed get) is cut into chunks of a launch-chosen size; warps stride over the chunks
// and never wait for one another.  Per chunk a warp
//   1. finds the row the chunk starts in with a 32-ary search of cu (one probe per lane and
//      round instead of a dependent bisection),
//   2. lets lane l resolve row r0 + l: its byte range on the packed side and where the row
//      lives on the other side (index -> tables), all lanes' lookups in flight together,
//   3. walks the rows, broadcasting each descriptor by shuffle, and copies the pieces that
//      fall inside the chunk as wide aligned vector traffic.
// With many resident warps per SM the metadata latency of one warp hides behind the copies of
// the others; there is no block-wide barrier on the path.
// --------------------------------------------------------------------------------------------
#ifndef TD_COPY_THREADS
#define TD_COPY_THREADS 256
#endif
constexpr int kCopyThreads = TD_COPY_THREADS;
constexpr int kCopyWarps = kCopyThreads / 32;
#ifndef TD_COPY_BLOCKS_PER_SM
#define TD_COPY_BLOCKS_PER_SM 2
#endif
#ifndef TD_CHUNK_TARGET_BYTES
#define TD_CHUNK_TARGET_BYTES 32768
#endif
constexpr int kCopyBlocksPerSM = TD_COPY_BLOCKS_PER_SM;      // resident CTAs per SM the copy kernels are built for
constexpr uint32_t kMinChunkBytes = 1024;                    // a warp is not given less than this
constexpr uint32_t kChunkTargetBytes = TD_CHUNK_TARGET_BYTES;   // chunk size aimed at when there is plenty of work

// All jobs of a launch (columns of a put, (request, column) pairs of a get) are laid end to end
// in one logical byte space, each job rounded up to 16 bytes.  The space is cut into chunks of
// equal size, chosen on the device from the actual total so that every warp of the grid gets
// the same whole number of chunks: balance over bytes is then exact whatever the mix of jobs
// and row lengths, and no chunk is left half empty at a job's end.
struct ChunkPlan {
    uint64_t chunk_bytes;    // multiple of 16
    uint64_t n_chunks;
};
__device__ __forceinline__ ChunkPlan plan_chunks(uint64_t total_bytes, uint64_t n_warps) {
    ChunkPlan p;
    const uint64_t per_warp = (total_bytes + n_warps - 1) / n_warps;
    // a warp with little to do takes it in two chunks from different parts of the space (rows
    // of different kinds cost differently), down to 8 KB each
    uint64_t target = per_warp / 2;
    if (target < 8192u) target = 8192u;
    if (target > kChunkTargetBytes) target = kChunkTargetBytes;
    uint64_t rounds = (per_warp + target / 2) / target;
    if (rounds < 1) rounds = 1;
    uint64_t c = (total_bytes + n_warps * rounds - 1) / (n_warps * rounds);
    c = (c + 15) & ~uint64_t(15);
    if (c < kMinChunkBytes) c = kMinChunkBytes;
    p.chunk_bytes = c;
    p.n_chunks = (total_bytes + c - 1) / c;
    return p;
}

// Chunks for a launch whose warps fetch them from a shared counter: about TD_DYN_CHUNKS_PER_WARP per
// warp, between 16 KB and 32 KB each.
#ifndef TD_DYN_CHUNKS_PER_WARP
#define TD_DYN_CHUNKS_PER_WARP 2
#endif
__device__ __forceinline__ ChunkPlan plan_chunks_dynamic(uint64_t total_bytes, uint64_t n_warps) {
    ChunkPlan p;
    uint64_t c = total_bytes / (n_warps * TD_DYN_CHUNKS_PER_WARP);
    c = (c + 15) & ~uint64_t(15);
#ifndef TD_DYN_MIN_CHUNK
#define TD_DYN_MIN_CHUNK 16384
#endif
    if (c < TD_DYN_MIN_CHUNK) {
        // a launch with less than 4 KB per warp is spread over as many warps as it has 4 KB
        // pieces (a micro-batch of a small shape: 12.3 -> 11.6 us); above that, fewer warps with
        // 16 KB each were measured faster than all warps with 8-13 KB
        c = total_bytes < n_warps * 4096u ? 4096u : TD_DYN_MIN_CHUNK;
    }
    if (c > 32768) c = 32768;
    p.chunk_bytes = c;
    p.n_chunks = (total_bytes + c - 1) / c;
    return p;
}

// Largest i in [0, rows) with key(i) <= x (the row holding position x, rows of no extent
// skipped); 0 when even key(0) > x.  Warp-cooperative; all lanes get the answer.
// Every load of a round is independent of the others, and the last round covers up to 256
// entries (eight per lane), so a table of up to 256 rows costs one memory round trip, one of up
// to 8192 rows two.  `along`, when given, is an array indexed like cu that the caller reads
// next (sample indices): its lines are prefetched into L1 beside the last round's loads.
// The key of row e is where it starts in the chunked space: cu[e] * esz + e * row_cost.
__device__ __forceinline__ uint32_t warp_find_row(const int32_t *cu, uint32_t rows, int64_t x, uint32_t esz,
                                                  uint32_t row_cost, uint32_t lane, const int32_t *along = nullptr) {
    uint32_t lo = 0, len = rows;
    while (len > 256u) {
        const uint32_t stride = (len + 31u) >> 5;
        const uint64_t probe = (uint64_t)lane * stride;
        const bool ok = probe < len &&
                        (int64_t)__ldg(cu + lo + probe) * esz + (int64_t)(lo + probe) * row_cost <= x;
        uint32_t cnt = __popc(__ballot_sync(kFullMask, ok));     // ok holds for a prefix of the lanes
        if (cnt < 1) cnt = 1;
        const uint32_t step = (cnt - 1u) * stride;
        lo += step;
        len = min(stride, len - step);
    }
    const uint32_t per = (len + 31u) >> 5;                       // entries per lane, at most 8
    const uint32_t e0 = lane * per;
    if (along && e0 < len) asm volatile("prefetch.global.L1 [%0];" ::"l"(along + lo + e0));
    uint32_t cnt = 0;
    #pragma unroll
    for (uint32_t t = 0; t < 8u; ++t)
        if (t < per && e0 + t < len &&
            (int64_t)__ldg(cu + lo + e0 + t) * esz + (int64_t)(lo + e0 + t) * row_cost <= x) ++cnt;
    cnt = __reduce_add_sync(kFullMask, cnt);                     // entries <= x form a prefix of the table
    return lo + (cnt ? cnt - 1u : 0u);
}

__device__ __forceinline__ uint64_t shfl_u64(uint64_t v, uint32_t src) {
    const uint32_t lo = __shfl_sync(kFullMask, (uint32_t)v, src);
    const uint32_t hi = __shfl_sync(kFullMask, (uint32_t)(v >> 32), src);
    return ((uint64_t)hi << 32) | lo;
}

__device__ __forceinline__ uint64_t shfl_up_u64(uint64_t v, int delta) {
    const uint32_t lo = __shfl_up_sync(kFullMask, (uint32_t)v, delta);
    const uint32_t hi = __shfl_up_sync(kFullMask, (uint32_t)(v >> 32), delta);
    return ((uint64_t)hi << 32) | lo;
}

// --------------------------------------------------------------------------------------------
// Asynchronous staging.  Each warp owns a ring of kStages shared-memory stages with one
// mbarrier each.  A piece of a row is fetched with one bulk asynchronous copy (cp.async.bulk,
// global to shared, completion counted in bytes on the stage's mbarrier); a piece is written
// out to its destination only when the ring is full and its stage is needed again, so a warp
// keeps kStages copies in flight, described by three warp-uniform registers each; the bytes
// in flight per SM are what a ragged copy needs to cover HBM latency, whatever the row
// lengths.  The bulk copy wants 16-byte aligned addresses and sizes:
// the source window is widened to the enclosing 16-byte boundaries (rows in an arena start
// aligned and are padded, so the window stays inside the arena) and the write-out shifts the
// bytes into place.  Every wait on an mbarrier is bounded; a warp that gives up records the
// error, falls back to plain loads and still drains its own copy before it returns.
// --------------------------------------------------------------------------------------------
#ifndef TD_STAGES
#define TD_STAGES 2
#endif
#ifndef TD_STAGE_BYTES
#define TD_STAGE_BYTES 6144
#endif
constexpr int kStages = TD_STAGES;
constexpr uint32_t kStageBytes = TD_STAGE_BYTES;
constexpr uint32_t kPieceMax = kStageBytes - 16;      // payload of one bulk copy; the aligned window still fits
// stages and mbarriers of one warp; rounded so that every warp's stages start 128-byte aligned
constexpr size_t kPipeSmemPerWarp = (((size_t)kStages * (kStageBytes + 8)) + 127) & ~size_t(127);
static_assert(kStageBytes % 16 == 0 && kPipeSmemPerWarp % 128 == 0, "bulk copies need 16-byte aligned stages");

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_global_to_shared(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

struct WarpPipe {
    uint32_t stage;            // shared-window address of this warp's kStages * kStageBytes bytes
    uint32_t bar;              // shared-window address of this warp's kStages mbarriers
    uint32_t parity;           // bit s: phase the next wait on stage s looks for
    uint32_t head, tail;       // copies issued / written out so far; stage of copy i is i % kStages
    uint32_t spin_limit;
    uint32_t failed;           // bit 0: a wait ran out, plain loads from here on; bit 1 + s: stage s may still be landing
    // the piece in flight in stage s (every lane holds the same values): destination, source
    // (the payload starts (source & 15) bytes into the stage), payload bytes
    uint8_t *p_dst[kStages];
    const uint8_t *p_src[kStages];
    uint32_t p_n[kStages];

    __device__ __forceinline__ void init(uint8_t *mem, uint32_t lane, uint32_t spin) {
        stage = smem_u32(mem);
        bar = stage + (uint32_t)kStages * kStageBytes;
        parity = 0; head = 0; tail = 0; spin_limit = spin; failed = 0;
        #pragma unroll
        for (int s = 0; s < kStages; ++s) { p_dst[s] = nullptr; p_src[s] = nullptr; p_n[s] = 0; }
        if (lane == 0) {
            for (int s = 0; s < kStages; ++s) mbar_init(bar + 8u * s, 1);
            fence_mbar_init();
        }
        __syncwarp();
    }

    __device__ __forceinline__ bool wait_stage(uint32_t s) {
        const uint32_t b = bar + 8u * s;
        const uint32_t ph = (parity >> s) & 1u;
        uint32_t polls = 0;
        bool ok = mbar_try_wait(b, ph);
        while (!ok && ++polls < spin_limit) { __nanosleep(20); ok = mbar_try_wait(b, ph); }
        if (ok) parity ^= 1u << s;
        return ok;
    }

    // write the oldest copy in flight out of its stage; if its wait runs out, redo it with plain loads
    __device__ __forceinline__ void drain_one(uint32_t lane) {
        const uint32_t s = tail % kStages;
        ++tail;
        uint8_t *dst = p_dst[0];
        const uint8_t *src = p_src[0];
        uint32_t n = p_n[0];
        #pragma unroll
        for (int i = 1; i < kStages; ++i)
            if (s == (uint32_t)i) { dst = p_dst[i]; src = p_src[i]; n = p_n[i]; }
        if (wait_stage(s)) {
            warp_copy_from_shared(dst, stage + s * kStageBytes + ((uint32_t)reinterpret_cast<uintptr_t>(src) & 15u), n, lane);
        } else {                                               // never seen; the piece is read again, directly
            failed |= 1u | (2u << s);
            warp_copy(dst, src, n, lane);
        }
    }

    // every copy issued so far written out to its destination
    __device__ __forceinline__ void drain_all(uint32_t lane) {
        while (tail != head) drain_one(lane);
    }

    // before the warp returns: everything written out, nothing of its own still landing
    __device__ __forceinline__ uint32_t finish(uint32_t lane) {
        while (tail != head) drain_one(lane);
        for (uint32_t s = 0; s < (uint32_t)kStages; ++s)
            if (failed & (2u << s)) wait_stage(s);
        return failed;
    }

    // Copy n bytes from src to dst through the stages (element-aligned, any length).  The bulk
    // copy reads the 16-byte aligned window around a piece; with kCheckWindow the window is
    // tested against [src_lo, src_hi) and a piece whose window would leave it is copied with
    // plain loads.  Arena rows start aligned and are padded to 16 bytes, so a get needs no test.
    template <bool kCheckWindow>
    __device__ __forceinline__ void push(uint8_t *dst, const uint8_t *src, uint32_t n, uint32_t lane,
                                         const uint8_t *src_lo, const uint8_t *src_hi) {
        while (n > 0) {
            uint32_t m = n > kPieceMax ? kPieceMax : n;
            const uint32_t pre = (uint32_t)(reinterpret_cast<uintptr_t>(src) & 15u);
            bool direct = failed || m < 64u;                             // after a failure, or too short to stage
            if (kCheckWindow && !direct) {
                // a window that would leave the buffer: only the few bytes at that edge go the
                // plain way, the piece is cut at the last 16-byte boundary inside the buffer
                if (src - pre < src_lo) {
                    m = min(m, 16u - pre);
                    direct = true;
                } else if (src - pre + ((pre + m + 15u) & ~15u) > src_hi) {
                    const uintptr_t last = reinterpret_cast<uintptr_t>(src_hi) & ~uintptr_t(15);
                    const uintptr_t at = reinterpret_cast<uintptr_t>(src);
                    if (last > at && last - at >= 64u) m = (uint32_t)(last - at);
                    else direct = true;                                  // fewer than 80 bytes are left
                }
            }
            const uint32_t size = (pre + m + 15u) & ~15u;
            if (direct) {
                warp_copy(dst, src, m, lane);
            } else {
                if (head - tail == (uint32_t)kStages) drain_one(lane);   // every stage busy: free the oldest
                const uint32_t s = head % kStages;
                ++head;
                #pragma unroll
                for (int i = 0; i < kStages; ++i)
                    if (s == (uint32_t)i) { p_dst[i] = dst; p_src[i] = src; p_n[i] = m; }
                __syncwarp();                                            // every lane is done reading stage s
                if (lane == 0) {
                    fence_proxy_async();
                    mbar_expect_tx(bar + 8u * s, size);
                    bulk_global_to_shared(stage + s * kStageBytes, src - pre, size, bar + 8u * s);
                }
            }
            dst += m; src += m; n -= m;
        }
    }
};

// The space that is cut into chunks charges every row of a ragged job a fixed kRowCost on top
// of its bytes, because that is what a row costs a warp (search, descriptor, a piece of its
// own): row i of a job takes [cu[i] * esz + i * kRowCost, cu[i+1] * esz + (i+1) * kRowCost),
// the fixed part first, its bytes behind it.  Chunks of equal size in this space take about
// equal time whether they hold a few long rows or many short ones.
#ifndef TD_ROW_COST
#define TD_ROW_COST 6144
#endif
constexpr uint32_t kRowCost = TD_ROW_COST;
static_assert(kRowCost % 16 == 0, "a job's extent stays a multiple of 16");

// Workflow step 3 for a put, row by row.  A row becomes visible to the controllers - its column
// bit set in the sample's status word, behind a fence - once all of it is in its arena.  A row
// that lies wholly inside one chunk is complete when that chunk's warp has written it out; a
// row that chunk borders cut is complete when the parts written by all the warps that share it
// add up to its length, which they count in progress[column][sample]; a row of no length
// belongs to the chunk that holds its place in the space.  Waiting for the ring to run empty
// and fencing after every chunk would cost more than the copying it interrupts, so a warp only
// notes what it has written (sample, column, elements, row length: one row per lane) and
// settles up to 32 notes at once: when the list is full, and when the warp is done.
struct PublishQueue {
    int32_t s;             // lane i: the i-th noted row's sample
    uint32_t part, total;  //         elements written by this warp / in the row
    uint32_t col;          //         its column
    uint32_t n;            // rows noted (the same in every lane)
};
__device__ __forceinline__ void publish_queue_init(PublishQueue &q) { q.s = -1; q.part = q.total = q.col = 0; q.n = 0; }

// Everything the warp has issued is written out and fenced; then the noted rows are settled.
__device__ __forceinline__ void publish_queue_flush(const DockView &dv, PublishQueue &q, WarpPipe &pipe, uint32_t lane) {
    if (q.n == 0) return;
    pipe.drain_all(lane);
    __threadfence();
    __syncwarp();
    bool ok = false;
    if (lane < q.n) {
        const uint32_t bit = 1u << q.col;
        bool complete = q.part == q.total;             // the whole row, or a row of no length
        if (!complete) {
            // the first time the count reaches the row's length (the same sample twice in one
            // call may push it beyond)
            const uint32_t old = atomicAdd(&dv.progress[(size_t)q.col * dv.n + (uint32_t)q.s], q.part);
            complete = old < q.total && old + q.part >= q.total;
            if (complete) __threadfence();
        }
        if (complete) ok = !(atomicOr(&dv.status[q.s], bit) & bit);
    }
    // accepted rows are counted per column: one addition per column the list holds
    const uint32_t live = __ballot_sync(kFullMask, lane < q.n);
    if (lane < q.n) {
        const uint32_t peers = __match_any_sync(live, q.col);
        const uint32_t okc = __popc(__ballot_sync(live, ok) & peers);
        if (okc && lane == (uint32_t)__ffs(peers) - 1u)
            atomicAdd(&dv.counters[CNT_PUT_ACCEPTED + q.col], (unsigned long long)okc);
    }
    q.n = 0;
}

// Notes the rows of one round: lanes with s_row >= 0 each hold one.
__device__ __forceinline__ void publish_queue_note(const DockView &dv, PublishQueue &q, WarpPipe &pipe, uint32_t lane,
                                                   int32_t s_row, uint32_t part, uint32_t total, uint32_t col) {
    const uint32_t m = __ballot_sync(kFullMask, s_row >= 0);
    const uint32_t cnt = __popc(m);
    if (cnt == 0) return;
    if (q.n + cnt > 32u) publish_queue_flush(dv, q, pipe, lane);
    // slot q.n + j takes the row of the j-th lane of m
    const uint32_t j = lane - q.n;                                  // meaningful for q.n <= lane < q.n + cnt
    const uint32_t src = (lane >= q.n && j < cnt) ? __fns(m, 0, (int)j + 1) : 0u;
    const int32_t s_in = __shfl_sync(kFullMask, s_row, src);
    const uint32_t part_in = __shfl_sync(kFullMask, part, src);
    const uint32_t total_in = __shfl_sync(kFullMask, total, src);
    if (lane >= q.n && j < cnt) { q.s = s_in; q.part = part_in; q.total = total_in; q.col = col; }
    q.n += cnt;
}

// Steps 2 and 3 for one chunk [b0, b1) of that space (a chunk is shorter than 4 GB) of a packed
// side described by cu[0..rows].  resolve(i, c0, c1, s) returns where row i starts on the other
// side, or nullptr to skip the row (and, for a put, the sample in s); it is called by one lane
// per row; `along` is the index array it reads (prefetched by the row search).  kToPacked: the
// packed side is the destination (get), else the source (put, whose source window is tested
// against the caller's buffer).  kPublish (put): the rows, or parts of rows, that the chunk
// holds are noted in `queue` for publication (see PublishQueue).
// seq_cu, when given, moves the rows on the packed side: row i then sits at element seq_cu[i]
// (seq_tail false) or ends at element seq_cu[i + 1] (seq_tail true) instead of starting at
// cu[i] - the two halves of a stream in which each sample's prompt row is followed by its
// response row; cu still says how long the rows are and where they lie in the chunked space.
struct NoAwait {
    __device__ __forceinline__ void operator()(uint32_t) const {}
};
template <bool kToPacked, bool kPublish, typename Resolve, typename Await = NoAwait>
__device__ __forceinline__ void warp_copy_chunk(const int32_t *cu, uint32_t rows, uint64_t b0, uint64_t b1,
                                                uint8_t *packed, uint32_t esz, uint32_t lane,
                                                const uint8_t *src_lo, const uint8_t *src_hi, WarpPipe &pipe,
                                                const int32_t *along, Resolve resolve,
                                                const int32_t *seq_cu = nullptr, bool seq_tail = false,
                                                const DockView *dvp = nullptr, PublishQueue *queue = nullptr,
                                                uint32_t column = 0, Await await = Await()) {
    uint32_t r0 = warp_find_row(cu, rows, (int64_t)b0, esz, kRowCost, lane, along);
    for (;;) {
        // lane l: the part of row r0 + l that falls inside the chunk, as (address on the packed
        // side, address on the other side, bytes); bytes = 0 when there is nothing to copy
        const uint32_t i = r0 + lane;
        bool in = false, wanted = false;
        uint32_t len = 0;
        uint8_t *mine = nullptr, *other = nullptr;
        int32_t s_row = -1;                // put: the sample of a row this lane has a part of, or owns
        uint32_t total = 0;                // put: the row's length in elements
        int64_t c0 = 0, c1 = 0;
        uint64_t dlo = 0, lo = 0, hi = 0;
        if (i < rows) {
            c0 = __ldg(cu + i);
            const uint64_t row0 = (uint64_t)c0 * esz + (uint64_t)i * kRowCost;
            in = c0 >= 0 && row0 < b1;
            if (in) {
                c1 = __ldg(cu + i + 1);
                dlo = row0 + kRowCost;                                       // the row's bytes, in the chunked space
                const uint64_t dhi = c1 > c0 ? dlo + (uint64_t)(c1 - c0) * esz : dlo;
                lo = max(dlo, b0); hi = min(dhi, b1);
                const bool empty_here = kPublish && c1 == c0 && row0 >= b0;   // a row of no length whose place is in this chunk
                wanted = hi > lo || empty_here;
            }
        }
        // rows inside the chunk form a prefix of the lanes
        const uint32_t n_rows = (uint32_t)__ffs(~__ballot_sync(kFullMask, in)) - 1u;   // 32 when all lanes are in
        await(r0 + n_rows);                // put: until the rows before that number have their places
        if (wanted) {
            int32_t s = -1;
            uint8_t *row = resolve(i, c0, c1, s);
            if (row) {
                s_row = s;
                total = (uint32_t)(c1 - c0);
                if (hi > lo) {
                    other = row + (lo - dlo);
                    uint64_t at = (uint64_t)c0;
                    if (seq_cu) at = seq_tail ? (uint64_t)((int64_t)__ldg(seq_cu + i + 1) - (c1 - c0))
                                              : (uint64_t)__ldg(seq_cu + i);
                    mine = packed + at * esz + (lo - dlo);
                    len = (uint32_t)(hi - lo);
                }
            }
        }
        uint32_t todo = __ballot_sync(kFullMask, len != 0);
        while (todo) {
            const uint32_t r = (uint32_t)__ffs(todo) - 1u;
            todo &= todo - 1u;
            const uint32_t len_r = __shfl_sync(kFullMask, len, r);
            uint8_t *p = reinterpret_cast<uint8_t *>(shfl_u64(reinterpret_cast<uint64_t>(mine), r));
            uint8_t *o = reinterpret_cast<uint8_t *>(shfl_u64(reinterpret_cast<uint64_t>(other), r));
            if (kToPacked) pipe.template push<false>(p, o, len_r, lane, src_lo, src_hi);
            else pipe.template push<true>(o, p, len_r, lane, src_lo, src_hi);
        }
        if (kPublish) publish_queue_note(*dvp, *queue, pipe, lane, s_row, len / esz, total, column);
        if (n_rows < 32u) break;
        r0 += 32u;
    }
}

}  // namespace td
