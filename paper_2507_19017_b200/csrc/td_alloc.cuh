// td_put, first kernel: reserve the rows of a put in the shard arenas.
// Workflow step 2 of "Distributed Transfer Dock Strategy" (a worker sends real data to the
// warehouses): before payload can move, every row needs its place.
#pragma once

#include "td_device.cuh"

namespace td {

constexpr int kAllocThreads = 1024;
constexpr int kAllocWarps = kAllocThreads / 32;
static_assert(kAllocWarps == 32, "the scan over the warps' sums gives one lane to each warp");
constexpr int kAllocPerMax = 4;                                // entries per thread and pass: 1, 2 or 4, by the size of the call
constexpr int kMaxPutItems = 8;                                // columns one put launch can carry
constexpr uint32_t kNotAllocating = 0xffffffffu;

struct PutArgs {
    uint32_t column, k;
    const int32_t *idx;
    const int32_t *cu;
    const uint8_t *data;
    uint64_t data_elems;
    const uint32_t *k_dev;                     // when set: the entry count, at most k, is read here on the device
};
// Entries of an item.  A worker that sends back what it computed from a batch does not know on
// the host how many samples the get returned; the count then comes from the get's result block.
__device__ __forceinline__ uint32_t item_k(const PutArgs &a) {
    return a.k_dev ? min(a.k, *a.k_dev) : a.k;
}
struct PutBatch {                              // the columns of one call, in call order
    uint32_t n_items;
    uint32_t pad;
    PutArgs item[kMaxPutItems];
    // follow[i] = 1 + the index of an earlier item of the same length class that item i may
    // ride along with in the alloc kernel (same entry count, not more data behind it), 0 = none.
    // The host only proposes; the kernel checks that the index and cu arrays are equal.
    uint8_t follow[kMaxPutItems];
    // A counter in the dock's workspace from which the scatter kernel hands out its chunks, private
    // to the stream the call was made on (calls on one stream run one after the other); nullptr:
    // every warp takes a fixed share instead.  Zeroed by the alloc kernel.
    unsigned long long *work_counter;
    // A word in the dock's workspace, private to the stream like the counter, in which the alloc
    // kernel stores `seq` (the call's number, growing from call to call) once everything ahead of
    // the call has finished: the scatter kernel, launched early, may read the call's inputs from
    // then on.  nullptr: the scatter kernel waits for the alloc kernel's end before it reads anything.
    unsigned long long *ready;
    unsigned long long seq;
    // Two more words behind `ready`, one per length class, when the call's followers are settled
    // on the host (progress != nullptr): the alloc kernel stores there, pass after pass, how
    // many entries of its class it has dealt with - counted over the class's leader items in call
    // order, tagged with the call's number - and the scatter kernel copies a row as soon as the
    // count has passed it, instead of waiting for the whole allocation.
    unsigned long long *progress;
};
__host__ __device__ __forceinline__ unsigned long long progress_pack(unsigned long long seq, uint32_t done) {
    return (seq << 32) | done;
}

static inline size_t put_alloc_smem_bytes(uint32_t S) {
    return (size_t)(kAllocWarps + 2) * S * sizeof(unsigned long long);
}

// Ordered exclusive prefix of `room` over the lanes that allocate in the same shard, and that
// shard's sum over the warp.  leader: the first allocating lane of its shard.
__device__ __noinline__ void warp_shard_prefix(bool alloc, uint32_t sh, uint32_t room, uint32_t lane,
                                                  unsigned long long &pre, unsigned long long &wsum, bool &leader) {
    pre = 0; wsum = 0; leader = false;
    const uint32_t mask = __ballot_sync(kFullMask, alloc);
    if (mask == 0) return;
    const uint32_t first = (uint32_t)__ffs(mask) - 1u;
    // usual case: every allocating lane of the warp is in one shard -> one shuffle scan
    const uint32_t first_sh = __shfl_sync(kFullMask, sh, first);      // every lane takes part
    if (__ballot_sync(kFullMask, alloc && sh != first_sh) == 0) {
        const uint32_t mine = alloc ? room : 0u;
        leader = alloc && lane == first;
        if (__ballot_sync(kFullMask, mine >> 26) == 0) {              // rows of the usual sizes: the warp's sum fits 32 bits
            uint32_t inc = mine;
            #pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t t = __shfl_up_sync(kFullMask, inc, d);
                if ((int)lane >= d) inc += t;
            }
            wsum = __shfl_sync(kFullMask, inc, 31);
            pre = inc - mine;
            return;
        }
        unsigned long long inc = mine;
        #pragma unroll 1
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long t = shfl_up_u64(inc, d);
            if ((int)lane >= d) inc += t;
        }
        wsum = shfl_u64(inc, 31);
        pre = inc - mine;
        return;
    }
    const uint32_t k2 = alloc ? sh : kNotAllocating;
    leader = alloc;
    #pragma unroll 1
    for (uint32_t j = 0; j < 32; ++j) {
        const uint32_t kj = __shfl_sync(kFullMask, k2, j);
        const uint32_t rj = __shfl_sync(kFullMask, room, j);
        if (alloc && kj == k2) {
            wsum += rj;
            if (j < lane) { pre += rj; leader = false; }
        }
    }
}

// Alloc.  grid = 2: CTA 0 serves the prompt-length items of the call, CTA 1 the response-length
// ones (the two classes share no table), each class's items one after the other, in passes of
// kAllocPass entries in call order.  Per pass:
//   1. every thread validates kAllocPer entries and settles with a CAS on len[] which of them
//      are first arrivals of their length class, i.e. reserve a row;
//   2. an ordered per-shard exclusive scan of the row sizes (every warp over its own run of
//      consecutive entries with shuffles, then the warps' sums through shared memory) gives
//      every new row the place, relative to the pass, a sequential walk would have given it;
//   3. one atomicAdd per shard reserves the pass's space; rows are placed behind it.
// A pass without a first arrival (a later column of a class whose rows exist) ends after 1.
// A pass that would overflow a shard is replayed by one thread, entry by entry, so that only
// the rows without room are refused.
// A worker that sends a whole record puts several columns of one length class for the same
// samples in the same order.  Such an item (a follower: its index and cu arrays equal those of
// an earlier item of the call, its leader) never reserves a row, and everything it has to be
// checked for follows from what the leader's thread already holds for the entry: the status
// word, the row length and the length in force after the leader's CAS.  Followers are therefore
// settled inside the leader's passes, without passes or atomics of their own.
// kAllocPer entries per thread and pass (a call of up to 1024 entries per length class runs the
// instance with one: a quarter of the code, which on a cold instruction cache is what counts).
template <int kAllocPer>
__global__ void __launch_bounds__(kAllocThreads)
put_alloc_kernel(const DockView dv, const PutBatch batch) {
    constexpr int kAllocPass = kAllocThreads * kAllocPer;          // entries per pass
    extern __shared__ unsigned long long smem_u64[];
    const uint32_t S = dv.S;
    unsigned long long *tot = smem_u64;                            // [kAllocWarps][S]
    unsigned long long *s_run = tot + (size_t)kAllocWarps * S;     // [S] space asked so far in this pass
    unsigned long long *s_start = s_run + S;                       // [S] where the pass's space begins
    __shared__ int32_t e_s[kAllocPass];
    __shared__ uint32_t e_room[kAllocPass];
    __shared__ uint8_t e_fok[kAllocPass];                          // bit f: follower f's entry was accepted
    __shared__ uint32_t s_overflow, s_not_following;

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t L = blockIdx.x + 1;                             // TD_PROMPT or TD_RESPONSE
    griddep_launch_dependents();                                   // the scatter may set itself up meanwhile
    const uint64_t cap = dv.cap[L];
    uint32_t n_oob = 0, n_dup = 0, n_bad = 0, n_mis = 0, n_full = 0;
    bool irregular = false;                    // a cu entry out of order or out of range, whatever else is wrong with its row

    // The passes read the items' index and cu arrays one after the other, each read at the head
    // of a chain of dependent accesses: ask for all of them now, one request per 128-byte line.
    for (uint32_t it = 0; it < batch.n_items; ++it) {
        const PutArgs &a = batch.item[it];
        if (dv.col_cls[a.column] != L) continue;
        const uint64_t bytes = (uint64_t)item_k(a) * 4u;
        for (uint64_t at = (uint64_t)tid * 128u; at < bytes; at += (uint64_t)kAllocThreads * 128u) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const uint8_t *>(a.idx) + at));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const uint8_t *>(a.cu) + at));
        }
    }

    // From here on the call's arrays and the dock's tables are read: whatever ran before this
    // kernel in the stream (a reset, the get whose batch is sent back, the caller's own producer)
    // must have finished.  The prefetch above only asked for lines.
    griddep_wait();
    if (blockIdx.x == 0 && tid == 0 && batch.work_counter) *batch.work_counter = 0;
    // Ahead of everything else: is every cu array of this class a non-decreasing sequence inside
    // its data?  The scatter kernel searches those arrays and must know before it starts; one
    // sweep over entries whose lines were asked for above.  Then the class reports its inputs
    // complete (the second class to do so makes the word read seq * 4 + 2).
    if (batch.ready) {
        #pragma unroll 1
        for (uint32_t it = 0; it < batch.n_items; ++it) {
            const PutArgs &a = batch.item[it];
            if (dv.col_cls[a.column] != L) continue;
            const uint32_t k = item_k(a);
            if (batch.follow[it] && a.cu == batch.item[batch.follow[it] - 1u].cu) {
                // the leader's very array, swept with the leader: only this item's own bound is left
                if (tid == 0 && k) irregular |= (uint64_t)a.cu[k] > a.data_elems;
                continue;
            }
            for (uint32_t i = tid; i < k; i += kAllocThreads) {
                const int64_t c0 = a.cu[i], c1 = a.cu[i + 1];
                irregular |= c1 < c0 || c0 < 0 || (uint64_t)c1 > a.data_elems;
            }
        }
        if (__syncthreads_or(irregular) && tid == 0) atomicOr(dv.errword, kErrIrregularCu);
        if (tid == 0) {
            __threadfence();
            atomicMax(batch.ready, batch.seq << 2);
            atomicAdd(batch.ready, 1ull);
        }
    }
    uint32_t done_before = 0;                  // entries of this class's earlier leader items

    // Which proposed followers really repeat their leader's index and cu arrays?  (Nothing to
    // find out, and no barrier to pass, when every one of them names its leader's own arrays.)
    bool to_compare = false;
    #pragma unroll 1
    for (uint32_t it = 0; it < batch.n_items; ++it)
        if (batch.follow[it] && dv.col_cls[batch.item[it].column] == L) {
            const PutArgs &a = batch.item[it], &ld = batch.item[batch.follow[it] - 1u];
            to_compare |= a.idx != ld.idx || a.cu != ld.cu;
        }
    uint32_t not_following = 0;
    if (to_compare) {
    if (tid == 0) s_not_following = 0;
    __syncthreads();
    {
        uint32_t differs = 0;
        #pragma unroll 1
        for (uint32_t it = 0; it < batch.n_items; ++it) {
            if (!batch.follow[it] || dv.col_cls[batch.item[it].column] != L) continue;
            const PutArgs &a = batch.item[it], &ld = batch.item[batch.follow[it] - 1u];
            if (a.idx == ld.idx && a.cu == ld.cu) continue;
            const uint32_t k = item_k(a);
            bool d = false;
            for (uint32_t i = tid; i <= k; i += kAllocThreads)
                d |= (i < k && a.idx[i] != ld.idx[i]) || a.cu[i] != ld.cu[i];
            if (d) differs |= 1u << it;
        }
        if (differs) atomicOr(&s_not_following, differs);
    }
    __syncthreads();
    not_following = s_not_following;
    // an item that does not follow after all takes its own passes, in its place in the call; so
    // do the later followers of its leader, which would otherwise overtake it
    #pragma unroll 1
    for (uint32_t it = 0; it < batch.n_items; ++it)
        if ((not_following >> it) & 1u)
            for (uint32_t f = it + 1; f < batch.n_items; ++f)
                if (batch.follow[f] == batch.follow[it]) not_following |= 1u << f;
    }

    #pragma unroll 1
    for (uint32_t it = 0; it < batch.n_items; ++it) {
        const PutArgs &a = batch.item[it];
        if (dv.col_cls[a.column] != L) continue;
        if (batch.follow[it] && !((not_following >> it) & 1u)) continue;      // settled with its leader
        uint32_t followers = 0;
        for (uint32_t f = it + 1; f < batch.n_items; ++f)
            if (batch.follow[f] == it + 1u && !((not_following >> f) & 1u)) followers |= 1u << f;
        const uint32_t bit = 1u << a.column;
        const uint32_t k = item_k(a);
        #pragma unroll 1
        for (uint32_t base = 0; base < k; base += kAllocPass) {
            // 1. validate, CAS.  A short pass is spread over all warps: each takes `per` rows of 32.
            //    A thread's entries go through the step side by side - their own words first,
            //    then every status word and CAS, then the verdicts - so that the dependent
            //    accesses of one entry do not wait for those of the one before.
            const uint32_t per = min((uint32_t)kAllocPer, (k - base + kAllocThreads - 1u) / kAllocThreads);
            int32_t s[kAllocPer];
            int64_t c0[kAllocPer], c1[kAllocPer];
            uint32_t room[kAllocPer], sh[kAllocPer], st[kAllocPer];
            int32_t old[kAllocPer];
            bool alloc[kAllocPer], have[kAllocPer], bad[kAllocPer];
            bool any = false;
            #pragma unroll
            for (int j = 0; j < kAllocPer; ++j) {
                // a warp owns 32 * per consecutive entries of the pass, in the order (j, lane)
                const uint32_t i = base + warp * (32u * per) + (uint32_t)j * 32u + lane;
                have[j] = (uint32_t)j < per && i < k;
                s[j] = -1; c0[j] = 0; c1[j] = 0;
                if (have[j]) { s[j] = a.idx[i]; c0[j] = a.cu[i]; c1[j] = a.cu[i + 1]; }
            }
            #pragma unroll
            for (int j = 0; j < kAllocPer; ++j) {
                st[j] = 0; old[j] = 0; bad[j] = false;
                if (!have[j]) continue;
                bad[j] = c1[j] < c0[j] || c0[j] < 0 || (uint64_t)c1[j] > a.data_elems;
                irregular |= bad[j];
                if (s[j] < 0 || (uint32_t)s[j] >= dv.n) continue;
                // The status word and the CAS travel side by side.  A column that is already
                // stored has its class's length set, so the CAS of a repeated put changes
                // nothing; it is then counted as a repeat, whatever its length says.
                st[j] = dv.status[s[j]];
                if (!bad[j]) old[j] = atomicCAS(&dv.len[L][s[j]], -1, (int32_t)(c1[j] - c0[j]));
            }
            #pragma unroll
            for (int j = 0; j < kAllocPer; ++j) {
                const uint32_t eo = warp * (32u * per) + (uint32_t)j * 32u + lane;
                alloc[j] = false; room[j] = 0; sh[j] = 0;
                if ((uint32_t)j >= per) continue;
                uint32_t fok = 0;
                if (have[j]) {
                    const int64_t l = c1[j] - c0[j];
                    if (s[j] < 0 || (uint32_t)s[j] >= dv.n) { ++n_oob; n_oob += __popc(followers); }
                    else {
                        if (st[j] & bit) { ++n_dup; }
                        else if (bad[j]) { ++n_bad; }
                        else if (old[j] == -1) {
                            alloc[j] = true;
                            room[j] = (uint32_t)align_row((uint64_t)l);
                            sh[j] = shard_of(dv, (uint32_t)s[j]);
                        } else if (old[j] != (int32_t)l) { ++n_mis; }
                        // Followers: same sample, same row.  Their bound on the data is not
                        // wider than the leader's, so where one of them is in order the leader
                        // has done its CAS and the length in force is known.
                        #pragma unroll 1
                        for (uint32_t fm = followers; fm; fm &= fm - 1u) {
                            const uint32_t f = (uint32_t)__ffs(fm) - 1u;
                            const PutArgs &b = batch.item[f];
                            if (st[j] & (1u << b.column)) ++n_dup;
                            else if (l < 0 || c0[j] < 0 || (uint64_t)c1[j] > b.data_elems) { ++n_bad; irregular = true; }
                            else if ((old[j] == -1 ? (int32_t)l : old[j]) != (int32_t)l) ++n_mis;
                            else fok |= 1u << f;
                        }
                    }
                }
                e_fok[eo] = (uint8_t)fok;
                e_s[eo] = s[j];
                e_room[eo] = alloc[j] ? room[j] : kNotAllocating;
                any |= alloc[j];
            }
            if (tid == 0) s_overflow = 0;
            if (__syncthreads_or(any)) {                          // else: no first arrival in this pass

            // 2. relative places: inside a warp its entries in order (four shuffle scans that
            //    carry the warp's per-shard sums along), then the warps in order (one scan over
            //    the warps' sums per shard)
            for (uint32_t q = lane; q < S; q += 32) tot[warp * S + q] = 0;
            __syncwarp();
            unsigned long long rel[kAllocPer];
            #pragma unroll
            for (int j = 0; j < kAllocPer; ++j) {
                rel[j] = 0;
                if ((uint32_t)j >= per) continue;                     // uniform
                unsigned long long pre, wsum;
                bool leader;
                warp_shard_prefix(alloc[j], sh[j], room[j], lane, pre, wsum, leader);
                rel[j] = alloc[j] ? tot[warp * S + sh[j]] + pre : 0ull;
                __syncwarp();
                if (leader) tot[warp * S + sh[j]] += wsum;
                __syncwarp();
            }
            __syncthreads();
            for (uint32_t k2 = warp; k2 < S; k2 += kAllocWarps) {
                const unsigned long long v = tot[lane * S + k2];
                unsigned long long inc = v;
                #pragma unroll 1
                for (int d = 1; d < 32; d <<= 1) {
                    const unsigned long long t = shfl_up_u64(inc, d);
                    if ((int)lane >= d) inc += t;
                }
                tot[lane * S + k2] = inc - v;                      // what the warps before this one ask for
                if (lane == 31) s_run[k2] = inc;                   // what the pass asks for
            }
            __syncthreads();
            #pragma unroll
            for (int j = 0; j < kAllocPer; ++j)
                if (alloc[j]) rel[j] += tot[warp * S + sh[j]];

            // 3. reserve the pass's space, place the rows
            for (uint32_t k2 = tid; k2 < S; k2 += kAllocThreads) {
                // rows of length zero still get a place: the cursor as it stands
                const unsigned long long start = atomicAdd(&dv.cursor[L][k2], s_run[k2]);
                if (start + s_run[k2] > cap) s_overflow = 1;
                s_start[k2] = start;
            }
            __syncthreads();
            if (!s_overflow) {
                #pragma unroll
                for (int j = 0; j < kAllocPer; ++j)
                    if (alloc[j]) dv.off[L][s[j]] = (long long)(s_start[sh[j]] + rel[j]);
            } else {
                // hand the pass's reservations back, then replay the pass in call order
                for (uint32_t k2 = tid; k2 < S; k2 += kAllocThreads)
                    atomicAdd(&dv.cursor[L][k2], 0ull - s_run[k2]);
                __syncthreads();
                if (tid == 0) {
                    const uint32_t n_here = min((uint32_t)kAllocPass, k - base);
                    for (uint32_t t = 0; t < n_here; ++t) {
                        const uint32_t r = e_room[t];
                        if (r == kNotAllocating) continue;
                        const int32_t ss = e_s[t];
                        const uint32_t k2 = shard_of(dv, (uint32_t)ss);
                        const unsigned long long start = atomicAdd(&dv.cursor[L][k2], (unsigned long long)r);
                        if (start + r > cap) {
                            atomicAdd(&dv.cursor[L][k2], 0ull - (unsigned long long)r);
                            atomicExch(&dv.len[L][ss], -1);
                            n_full += 1u + __popc((uint32_t)e_fok[t]);      // its followers find no row either
                        } else {
                            dv.off[L][ss] = (long long)start;
                        }
                    }
                }
            }
            __syncthreads();
            }
            // the rows of this pass have their places: whoever copies them may go ahead
            if (batch.progress && tid == 0) {
                __threadfence();
                st_release_u64(&batch.progress[L - 1],
                               progress_pack(batch.seq, done_before + min(base + (uint32_t)kAllocPass, k)));
            }
        }
        done_before += k;
    }
    n_oob = __reduce_add_sync(kFullMask, n_oob);
    n_dup = __reduce_add_sync(kFullMask, n_dup);
    n_bad = __reduce_add_sync(kFullMask, n_bad);
    n_mis = __reduce_add_sync(kFullMask, n_mis);
    n_full = __reduce_add_sync(kFullMask, n_full);
    irregular = __any_sync(kFullMask, irregular);
    if (lane == 0) {
        // the scatter kernel of this call, and of later ones until a reset, then takes rows one by one
        if (irregular) atomicOr(dv.errword, kErrIrregularCu);
        if (n_oob) flag_error(dv, TD_ERR_OOB_INDEX, CNT_OOB, n_oob);
        if (n_dup) flag_error(dv, TD_ERR_DUP_PUT, CNT_DUP, n_dup);
        if (n_bad) flag_error(dv, TD_ERR_BAD_LENGTH, CNT_BADLEN, n_bad);
        if (n_mis) flag_error(dv, TD_ERR_LEN_MISMATCH, CNT_MISMATCH, n_mis);
        if (n_full) flag_error(dv, TD_ERR_ARENA_FULL, CNT_FULL, n_full);
    }
}

}  // namespace td
