// Device-side view of a dock and the warp-level ragged copy shared by put and get.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/td.h"

namespace td {

constexpr int kMaxColumns = 32;
constexpr uint32_t kRowAlign = 8;            // rows start on multiples of 8 elements (>= 16 bytes)
constexpr uint32_t kFullMask = 0xffffffffu;

// counters[] slots (uint64 each)
enum : int {
    CNT_PUT_ACCEPTED = 0,    // + column
    CNT_GOT_SAMPLES = 32,    // + consumer
    CNT_GOT_TOKENS = 64,     // + consumer
    CNT_OOB = 96, CNT_DUP, CNT_MISMATCH, CNT_FULL, CNT_TRUNC, CNT_BADLEN, CNT_CONFLICT, CNT_TIMEOUT,
    CNT_TOTAL = 112
};

// Everything a kernel needs to know about a dock; passed by value (constant bank).
struct DockView {
    uint32_t G, N, S, n;
    uint32_t ncol, ncons;
    uint32_t prompts_per_shard;
    uint32_t reward_col;
    uint32_t claim_words, consumed_words;   // words per consumer
    uint32_t spin_limit;                    // polls before a look-back wait gives up
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
    uint8_t  *colbase[kMaxColumns];         // arena (S * cap * esz) or scalar store (n * esz)
    uint32_t need[kMaxColumns];             // per consumer
    uint32_t outm[kMaxColumns];
    uint32_t cflags[kMaxColumns];
    uint32_t col_pad[kMaxColumns];
    uint8_t  col_esz[kMaxColumns];
    uint8_t  col_cls[kMaxColumns];
};

__device__ __forceinline__ uint32_t shard_of(const DockView &dv, uint32_t s) {
    return (s / dv.N) / dv.prompts_per_shard;
}

__device__ __forceinline__ uint64_t align_row(uint64_t elems) {
    return (elems + (kRowAlign - 1)) & ~uint64_t(kRowAlign - 1);
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
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

__device__ __forceinline__ void flag_error(const DockView &dv, uint32_t bit, int counter, uint32_t count = 1) {
    atomicOr(dv.errword, bit);
    atomicAdd(&dv.counters[counter], (unsigned long long)count);
}

// --------------------------------------------------------------------------------------------
// Warp-cooperative copy of nbytes from src to dst.  Both are aligned to the element size
// (2 or 4 bytes) and nbytes is a multiple of it; nothing else is assumed.  Stores are issued
// as aligned 16-byte vectors; the source stream is read as aligned 16-byte vectors too and
// shifted into place when the two sides disagree modulo 16.  [src_lo, src_hi) bounds the
// buffer the source lies in: an aligned source vector that would reach outside it is
// assembled from element loads instead.
// --------------------------------------------------------------------------------------------
__device__ __forceinline__ void copy_elems(uint8_t *dst, const uint8_t *src, uint32_t count,
                                           uint32_t esz, uint32_t lane) {
    // count < 32 elements
    if (lane < count) {
        if (esz == 4)
            reinterpret_cast<uint32_t *>(dst)[lane] = reinterpret_cast<const uint32_t *>(src)[lane];
        else
            reinterpret_cast<uint16_t *>(dst)[lane] = reinterpret_cast<const uint16_t *>(src)[lane];
    }
}

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4 *p, uint4 v) { __stcs(p, v); }

// 16 source bytes starting `delta` bytes into the 32-byte window (a, b); delta in 2..14, even.
template <int WSH>
__device__ __forceinline__ uint4 shift_window(const uint4 &a, const uint4 &b, uint32_t bsh) {
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint4 r;
    r.x = __funnelshift_r(w[WSH + 0], w[WSH + 1], bsh);
    r.y = __funnelshift_r(w[WSH + 1], w[WSH + 2], bsh);
    r.z = __funnelshift_r(w[WSH + 2], w[WSH + 3], bsh);
    r.w = __funnelshift_r(w[WSH + 3], w[(WSH + 4) & 7], bsh);   // w[WSH+4] is only used when bsh > 0
    return r;
}

__device__ __forceinline__ uint4 load_window_slow(const uint8_t *p, uint32_t esz) {
    // 16 bytes from an element-aligned address, element by element
    uint4 r;
    if (esz == 4) {
        const uint32_t *q = reinterpret_cast<const uint32_t *>(p);
        r.x = q[0]; r.y = q[1]; r.z = q[2]; r.w = q[3];
    } else {
        const uint16_t *q = reinterpret_cast<const uint16_t *>(p);
        r.x = q[0] | (uint32_t(q[1]) << 16); r.y = q[2] | (uint32_t(q[3]) << 16);
        r.z = q[4] | (uint32_t(q[5]) << 16); r.w = q[6] | (uint32_t(q[7]) << 16);
    }
    return r;
}

template <int WSH>
__device__ __forceinline__ void copy_body_shifted(uint4 *dst, const uint8_t *src, uint32_t nvec,
                                                  uint32_t delta, uint32_t esz, uint32_t lane,
                                                  const uint8_t *src_lo, const uint8_t *src_hi) {
    const uint4 *S = reinterpret_cast<const uint4 *>(src - delta);
    const uint32_t bsh = (delta & 3u) * 8u;
    // vectors whose 32-byte window lies inside [src_lo, src_hi)
    uint32_t v_lo = 0, v_hi = nvec;
    if (reinterpret_cast<const uint8_t *>(S) < src_lo) v_lo = 1;
    if (reinterpret_cast<const uint8_t *>(S + nvec + 1) > src_hi) v_hi = nvec - 1;
    if (lane == 0) {
        if (v_lo == 1) st_stream(dst, load_window_slow(src, esz));
        if (v_hi != nvec && nvec >= 1 && !(v_lo == 1 && nvec == 1))
            st_stream(dst + (nvec - 1), load_window_slow(src + 16ull * (nvec - 1), esz));
    }
    if (v_hi <= v_lo) return;
    uint32_t v = v_lo + lane;
    for (; v + 96 < v_hi; v += 128) {
        uint4 a0 = ld_stream(S + v),      b0 = ld_stream(S + v + 1);
        uint4 a1 = ld_stream(S + v + 32), b1 = ld_stream(S + v + 33);
        uint4 a2 = ld_stream(S + v + 64), b2 = ld_stream(S + v + 65);
        uint4 a3 = ld_stream(S + v + 96), b3 = ld_stream(S + v + 97);
        st_stream(dst + v,      shift_window<WSH>(a0, b0, bsh));
        st_stream(dst + v + 32, shift_window<WSH>(a1, b1, bsh));
        st_stream(dst + v + 64, shift_window<WSH>(a2, b2, bsh));
        st_stream(dst + v + 96, shift_window<WSH>(a3, b3, bsh));
    }
    for (; v < v_hi; v += 32) {
        uint4 a = ld_stream(S + v), b = ld_stream(S + v + 1);
        st_stream(dst + v, shift_window<WSH>(a, b, bsh));
    }
}

__device__ __forceinline__ void warp_copy(uint8_t *dst, const uint8_t *src, uint64_t nbytes,
                                          uint32_t esz, uint32_t lane,
                                          const uint8_t *src_lo, const uint8_t *src_hi) {
    if (nbytes == 0) return;
    // head: bring dst to a 16-byte boundary
    uint32_t head = (16u - (uint32_t)(reinterpret_cast<uintptr_t>(dst) & 15u)) & 15u;
    if (head > nbytes) head = (uint32_t)nbytes;
    if (head) {
        copy_elems(dst, src, head / esz, esz, lane);
        dst += head; src += head; nbytes -= head;
    }
    const uint32_t nvec = (uint32_t)(nbytes >> 4);
    const uint32_t delta = (uint32_t)(reinterpret_cast<uintptr_t>(src) & 15u);
    if (nvec) {
        uint4 *D = reinterpret_cast<uint4 *>(dst);
        if (delta == 0) {
            const uint4 *S = reinterpret_cast<const uint4 *>(src);
            uint32_t v = lane;
            for (; v + 96 < nvec; v += 128) {
                uint4 a0 = ld_stream(S + v), a1 = ld_stream(S + v + 32);
                uint4 a2 = ld_stream(S + v + 64), a3 = ld_stream(S + v + 96);
                st_stream(D + v, a0); st_stream(D + v + 32, a1);
                st_stream(D + v + 64, a2); st_stream(D + v + 96, a3);
            }
            for (; v < nvec; v += 32) st_stream(D + v, ld_stream(S + v));
        } else {
            switch (delta >> 2) {
                case 0: copy_body_shifted<0>(D, src, nvec, delta, esz, lane, src_lo, src_hi); break;
                case 1: copy_body_shifted<1>(D, src, nvec, delta, esz, lane, src_lo, src_hi); break;
                case 2: copy_body_shifted<2>(D, src, nvec, delta, esz, lane, src_lo, src_hi); break;
                default: copy_body_shifted<3>(D, src, nvec, delta, esz, lane, src_lo, src_hi); break;
            }
        }
    }
    const uint32_t tail = (uint32_t)(nbytes & 15u);
    if (tail) copy_elems(dst + 16ull * nvec, src + 16ull * nvec, tail / esz, esz, lane);
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
    for (uint64_t v = lane; v < nvec; v += 32) st_stream(D + v, val);
    const uint32_t tail = (uint32_t)(nbytes & 15u);
    if (tail && lane < tail / esz) {
        uint8_t *t = dst + 16ull * nvec;
        if (esz == 4) reinterpret_cast<uint32_t *>(t)[lane] = bits;
        else reinterpret_cast<uint16_t *>(t)[lane] = (uint16_t)bits;
    }
}

// --------------------------------------------------------------------------------------------
// Span copy.  The packed side of a ragged copy (the source of a put, the destination of a
// packed get) is cut into spans of kSpanBytes; one CTA serves one span at a time:
//   1. all threads together find the row the span starts in (a k-ary search of cu with one
//      probe per thread and round, instead of a dependent bisection per warp);
//   2. one thread per row resolves where that row lives on the other side (index -> tables);
//   3. each warp copies its kWarpBytes slice of the span, piece by piece, from the row
//      descriptors now in shared memory.
// This keeps every dependent metadata lookup off the warps' critical path and leaves the
// copy itself as wide aligned vector traffic.
// --------------------------------------------------------------------------------------------
constexpr int kSpanThreads = 256;
constexpr int kSpanWarps = kSpanThreads / 32;
constexpr uint32_t kWarpBytes = 4096;
constexpr uint32_t kSpanBytes = kWarpBytes * kSpanWarps;

struct RowDesc {
    uint64_t lo, hi;          // byte range of the row on the packed side
    uint8_t *other;           // start of the row on the other side, nullptr = skip the row
};

// Largest i in [0, rows) with cu[i] <= x (the row holding element x, rows of length zero
// skipped); 0 when even cu[0] > x.  Every thread of the CTA must call it; all get the answer.
__device__ __forceinline__ uint32_t block_find_row(const int32_t *cu, uint32_t rows, int64_t x) {
    uint32_t lo = 0, len = rows;
    while (len > 1) {
        const uint32_t stride = (len + kSpanThreads - 1) / kSpanThreads;
        const uint64_t probe = (uint64_t)threadIdx.x * stride;
        const bool ok = probe < len && (int64_t)cu[lo + probe] <= x;
        int cnt = __syncthreads_count(ok);          // ok holds for a prefix of the threads
        if (cnt < 1) cnt = 1;
        const uint32_t step = (uint32_t)(cnt - 1) * stride;
        lo += step;
        len = min(stride, len - step);
    }
    return lo;
}

// First descriptor in d[0, n) whose hi exceeds x (hi is non-decreasing); n if none.
__device__ __forceinline__ uint32_t first_desc_after(const RowDesc *d, uint32_t n, uint64_t x) {
    uint32_t lo = 0, hi = n;
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if (d[mid].hi > x) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// Step 3 for one warp: copy the parts of the described rows that fall inside [w_lo, w_hi) of
// the packed side.  kToPacked: the packed side is the destination (get), else the source (put).
template <bool kToPacked>
__device__ __forceinline__ void warp_copy_rows(const RowDesc *d, uint32_t n, uint64_t w_lo, uint64_t w_hi,
                                               uint8_t *packed, uint32_t esz, uint32_t lane,
                                               const uint8_t *src_lo, const uint8_t *src_hi) {
    for (uint32_t r = first_desc_after(d, n, w_lo); r < n; ++r) {
        const uint64_t rlo = d[r].lo;
        if (rlo >= w_hi) break;
        uint8_t *other = d[r].other;
        if (other == nullptr) continue;
        const uint64_t lo = max(rlo, w_lo), hi = min(d[r].hi, w_hi);
        if (hi <= lo) continue;
        if (kToPacked) warp_copy(packed + lo, other + (lo - rlo), hi - lo, esz, lane, src_lo, src_hi);
        else warp_copy(other + (lo - rlo), packed + lo, hi - lo, esz, lane, src_lo, src_hi);
    }
}

}  // namespace td
