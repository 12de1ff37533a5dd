/*
 * td.h - C ABI of the transfer dock: put/get dispatch of RL samples held in GPU memory.
 *
 * The dock follows the sample flow of "Distributed Transfer Dock Strategy" (Fig. 4, Eq. 4):
 *   warehouses  hold the real data, the buffer being split along the global batch with every
 *               sample keeping its own index        -> per-column ragged arenas, S shards;
 *   controllers (one per worker state) record which samples that state may still be served
 *                                                   -> per-consumer claim / consumed bitmaps;
 *   workflow    1. a worker state asks its controller for metadata     (td_get: select)
 *               2. it fetches, or sends, the real data                 (td_get: gather, td_put)
 *               3. the warehouse updates its state, visible to every controller
 *                                                                      (td_put: publish).
 * The record schema is the one under Eq. 1: one prompt-length item, several response-length
 * items and a few scalars per sample; samples come in GRPO groups of N responses per prompt
 * (Fig. 2).  The group-normalised advantage is not given in the paper; td_get computes
 * A = (r - mean) / (std + eps) over each dispatched group, population std, in double.
 *
 * Conventions for every call:
 *   - "device" pointers are CUDA device memory owned by the caller; the library allocates no
 *     device memory and frees none.  "host" pointers are ordinary host memory.  The one
 *     allocation the library makes is pinned HOST memory: td_get_many_host with a staging
 *     buffer allocates a host mirror of it once per plan (freed by td_plan_destroy).
 *   - td_put / td_get / td_get_many / td_reset only enqueue work on the given stream and return;
 *     they never synchronise.  Calls on one stream execute in call order.  Gets may run
 *     concurrently with each other and with puts on other streams.  Puts that may reserve the
 *     same row (the first columns of a length class to arrive for a sample) must be ordered by
 *     the caller; puts of further columns for samples whose rows of that class are stored and
 *     published (the write-backs of worker states) only read the tables and may overlap.
 *   - return value: TD_OK (0) or a negative td_error found on the host.  Conditions found on the
 *     device never trap: the offending sample is skipped, a TD_ERR_* bit is OR-ed into the
 *     dock's error word (td_status) and, for a get, into td_result.status.
 *   - a streamlike argument is a cudaStream_t passed as void* (NULL = the default stream).
 */
#ifndef TD_H
#define TD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct td_dock td_dock;          /* opaque host object */

enum { TD_I32 = 0, TD_F32 = 1, TD_BF16 = 2 };             /* td_column.dtype */
enum { TD_SCALAR = 0, TD_PROMPT = 1, TD_RESPONSE = 2 };   /* td_column.cls   */
enum { TD_PACKED = 0, TD_PADDED = 1 };                    /* td_get_out.mode */
enum { TD_OUT_LEFT_PAD_PROMPT = 1u };                     /* td_get_out.flags */
enum { TD_F_ADVANTAGE = 1u };                             /* td_consumer.flags */

typedef enum {
    TD_OK = 0,
    TD_EINVAL = -1,       /* bad argument                                   */
    TD_EWORKSPACE = -2,   /* workspace or scratch too small or misaligned   */
    TD_ECUDA = -3,        /* a CUDA runtime call failed (no device, ...)    */
    TD_ETOOLARGE = -4     /* td_get_static: the dock exceeds its fixed scratch */
} td_error;

/* device-detected conditions */
enum {
    TD_ERR_OOB_INDEX        = 1u << 0,  /* put: sample index outside [0, G*N)                  */
    TD_ERR_DUP_PUT          = 1u << 1,  /* put: (sample, column) already stored; first one kept */
    TD_ERR_LEN_MISMATCH     = 1u << 2,  /* put: length differs from the sample's length class   */
    TD_ERR_ARENA_FULL       = 1u << 3,  /* put: shard arena has no room for the row             */
    TD_ERR_OUT_TRUNCATED    = 1u << 4,  /* get: stopped before a group that would not fit       */
    TD_ERR_LOOKBACK_TIMEOUT = 1u << 5,  /* get: a scan tile gave up waiting; nothing is served,
                                           nothing stays claimed, the groups remain available   */
    TD_ERR_BAD_LENGTH       = 1u << 6,  /* put: cu not monotone or beyond data_elems            */
    TD_ERR_COPY_TIMEOUT     = 1u << 7   /* a staged copy did not land in time; plain loads used  */
};

typedef struct {
    const char *name;      /* not kept */
    int32_t  dtype;        /* TD_I32 | TD_F32 | TD_BF16; payload is copied as raw bits */
    int32_t  cls;          /* TD_SCALAR: one element per sample; TD_PROMPT / TD_RESPONSE:
                              a row whose length is the sample's prompt / response length */
    uint32_t pad_bits;     /* raw bit pattern written behind a row in TD_PADDED mode */
} td_column;

typedef struct {
    const char *name;      /* not kept */
    uint32_t need_mask;    /* bit c: column c must be stored before a sample is served */
    uint32_t out_mask;     /* bit c: column c is gathered; must lie within need_mask   */
    uint32_t flags;        /* TD_F_ADVANTAGE: needs reward_column within need_mask     */
} td_consumer;

typedef struct {
    uint32_t n_prompts;    /* G */
    uint32_t n_per_group;  /* N; sample s = prompt * N + response, group = s / N; G * N < 2^30 */
    uint32_t n_shards;     /* S warehouses, 1..256, must divide G; shard(s) = (s / N) / (G / S) */
    uint32_t n_columns;    const td_column   *columns;     /* 1..32, host array */
    uint32_t n_consumers;  const td_consumer *consumers;   /* 1..32, host array */
    uint64_t prompt_elems_per_shard;    /* arena capacity per shard, elements (rounded up to 8) */
    uint64_t response_elems_per_shard;
    uint32_t reward_column;             /* a TD_F32 TD_SCALAR column */
    float    adv_eps;
    int32_t  device;                    /* CUDA device ordinal of the workspace */
} td_config;

/* Written by td_get on the device; read it after the stream has reached that point. */
typedef struct {
    uint32_t n_samples, n_groups;             /* n_samples = n_groups * N */
    uint64_t prompt_tokens, response_tokens;  /* = cu_prompt[n_samples], cu_response[n_samples] */
    uint32_t status;                          /* TD_ERR_* bits of this call */
    uint32_t reserved;
} td_result;

/* Output buffers of one get.  The struct itself is host memory; every pointer in it is
 * caller-owned DEVICE memory that stays valid until the get has executed.  The payload buffers
 * (col[], seq, seq_advantages) may instead be page-locked host memory that the device can
 * address (cudaHostAlloc / cudaHostRegister under unified addressing): the gather then writes
 * the batch across the bus itself, in wide contiguous stores, and a worker whose tensors live on
 * the host needs no copy afterwards.  indices, the cu arrays, advantages and result are read
 * back by the kernels and belong in device memory. */
typedef struct {
    int32_t  mode;                    /* TD_PACKED: column c holds its rows back to back, row i at
                                         cu_<class>[i]; TD_PADDED: row i at i * pad_<class>_to,
                                         filled up with the column's pad_bits */
    uint32_t pad_prompt_to, pad_response_to;   /* row widths in elements (TD_PADDED only) */
    uint32_t flags;                   /* 0, or TD_OUT_LEFT_PAD_PROMPT: in TD_PADDED mode a row of a
                                         TD_PROMPT column ends at its width, (pad_prompt_to - length)
                                         copies of pad_bits in front of it, so that in a dense
                                         [prompt | response] batch every response starts at the same
                                         position, as batched generation lays its sequences out;
                                         TD_RESPONSE rows are padded behind as always, TD_PACKED
                                         ignores the flag.  Any other bit: TD_EINVAL */
    int32_t *indices;                 /* [max_samples] sample indices, ascending          required */
    int32_t *cu_prompt, *cu_response; /* [max_samples + 1] prefix sums of the true lengths required */
    int32_t *cu_seq;                  /* [max_samples + 1] cu_prompt + cu_response, or NULL */
    void    *col[32];                 /* per column; NULL = not wanted                     */
    uint64_t col_capacity_elems[32];  /* room behind col[c], in elements                   */
    float   *advantages;              /* [max_samples]; required iff TD_F_ADVANTAGE        */
    td_result *result;                /* required                                          */
    void    *scratch;                 /* td_get_scratch_bytes() bytes, 16-byte aligned, private to
                                         this call while it is in flight; zero-filled once after
                                         allocation, never needs clearing afterwards       required */
    uint64_t scratch_bytes;
    /* Fused token stream, optional (seq == NULL and seq_advantages == NULL: not wanted; a zeroed
     * struct asks for neither).  What a varlen trainer reads directly: sample i's row of column
     * seq_prompt_col (TD_PROMPT) followed by its row of column seq_response_col (TD_RESPONSE, same
     * element size, both within the consumer's out_mask) at element cu_seq[i] of `seq`, in
     * either output mode; cu_seq is then required.  seq_advantages (needs TD_F_ADVANTAGE) has the
     * same layout in float: 0 on prompt tokens, the sample's advantage on its response tokens,
     * i.e. advantage times loss mask.  seq_capacity_elems is the room behind each of the two; a
     * group that would not fit ends the batch (TD_ERR_OUT_TRUNCATED). */
    uint32_t seq_prompt_col, seq_response_col;
    void    *seq;
    uint64_t seq_capacity_elems;
    float   *seq_advantages;
} td_get_out;

typedef struct {
    uint64_t put_accepted[32];        /* per column */
    uint64_t got_samples[32];         /* per consumer */
    uint64_t got_tokens[32];          /* per consumer, prompt + response tokens */
    uint64_t n_oob, n_dup, n_len_mismatch, n_arena_full, n_truncated, n_bad_length;
    uint64_t n_claim_conflicts;       /* groups lost to a concurrent get of the same consumer */
    uint64_t n_lookback_timeouts;
    uint32_t error_word;              /* OR of all TD_ERR_* bits since the last reset */
    uint32_t reserved;
} td_stats;

/* Bytes of device workspace a dock with this configuration needs (tables, bitmaps and the
 * arenas of Eq. 4's payload term).  Host only; no CUDA call. */
int td_query_workspace(const td_config *cfg, size_t *bytes);

/* Builds a dock inside `d_workspace` (device, 256-byte aligned, `bytes` >= td_query_workspace)
 * and brings it to the empty state on the default stream, synchronising once.  The workspace
 * stays the caller's and must outlive the dock.  *out is freed by td_destroy. */
int td_create(const td_config *cfg, void *d_workspace, size_t bytes, td_dock **out);
int td_destroy(td_dock *dock);

/* Workflow steps 2 and 3 for a producer: store column `column` of the k samples d_indices[0..k)
 * and make them visible to every consumer.
 *   d_indices  device int32 [k], any order.
 *   d_cu       device int32 [k + 1], non-decreasing element offsets of the rows inside d_data;
 *              NULL for a TD_SCALAR column (row i is element i).
 *   d_data     device, rows back to back, data_elems elements in total (bounds what is read).
 * Rows are placed in call order: the first column of a length class to arrive for a sample
 * fixes its length and reserves its row at the next free element of the sample's shard.
 * Samples that are out of range, already stored, of the wrong length or without room are
 * skipped and counted.  The same index twice within one call is safe but leaves that row's
 * content unspecified. */
int td_put(td_dock *dock, uint32_t column, const int32_t *d_indices, uint32_t k,
           const int32_t *d_cu, const void *d_data, uint64_t data_elems, void *stream);

/* Workflow steps 1 and 2 for worker state `consumer`: claim the lowest-numbered groups whose
 * need_mask columns are all stored and that this consumer has not been served, at most
 * max_samples / N of them, and gather their out_mask columns, cu_seqlens and (TD_F_ADVANTAGE)
 * advantages into `out`.  Fewer groups than asked for, zero included, is not an error.  The
 * batch ends before the first group that would overflow a supplied buffer (TD_ERR_OUT_TRUNCATED;
 * that group stays available).  A group is never served twice to one consumer, also when gets
 * of that consumer run concurrently on several streams; such a get may then return fewer
 * groups than were ready. */
int td_get(td_dock *dock, uint32_t consumer, uint32_t max_samples, const td_get_out *out,
           void *stream);
size_t td_get_scratch_bytes(const td_dock *dock);

/* td_get for callers that cannot provide scratch memory.  (The paper has no counterpart: this
 * is a convenience of this library.)  Some code that wants to serve a batch may not allocate
 * device memory at all: a step running inside a serving loop whose memory pool is frozen, a
 * plug-in that is handed nothing but its input and output buffers, a process whose memory
 * budget is already committed.  td_get asks such a caller for td_get_scratch_bytes() of
 * zero-filled device memory it does not have.  td_get_static does the same get with the scan
 * scratch kept in a fixed array inside the library (about 65 KB, held by every GPU that loads
 * the library until the process exits); out->scratch and out->scratch_bytes are ignored, every
 * other field of `out` means what it means for td_get, and the results are the same.
 *   - Limit: docks of at most 16384 prompts (G); a larger dock gets TD_ETOOLARGE and nothing
 *     is enqueued.
 *   - The call allocates and frees nothing.  Its first call on a device looks the array's device
 *     address up (once per device; a host-side query, no allocation); make that first call
 *     outside any stream capture.
 *   - All calls share the one array, which still holds the previous call's contents; the words
 *     that must start at zero are cleared on `stream` before the scan.  Two td_get_static calls
 *     that overlap on the GPU (different streams, no ordering between them) race on it: they
 *     share the scan's ticket, its tile descriptors and its candidate list, so the outcome is
 *     undefined within the dock's own tables: either call may return nothing, report
 *     TD_ERR_LOOKBACK_TIMEOUT, be served groups that the other call selected (also groups of
 *     the other call's consumer, whose served marks are then set for the wrong worker state),
 *     or leave groups claimed and unserved until td_reset.  No memory outside the dock, the
 *     array and the two calls' own output buffers is touched.  Order such calls (one stream,
 *     or events), or use td_get with separate scratch for gets that may overlap. */
int td_get_static(td_dock *dock, uint32_t consumer, uint32_t max_samples, const td_get_out *out,
                  void *stream);

/* Several columns in one call, as a worker that sends a whole record does (prompt and response
 * ids together, say): the items are stored as if td_put had been called on each in array order,
 * with three kernel launches for up to eight items instead of three per item.  Every field of
 * an item means what the td_put argument of the same name means. */
typedef struct {
    uint32_t column, k;
    const int32_t *d_indices;
    const int32_t *d_cu;
    const void *d_data;
    uint64_t data_elems;
} td_put_item;
int td_put_many(td_dock *dock, const td_put_item *items, uint32_t n_items, void *stream);

/* Workflow steps 2 and 3 for a worker state that sends back what it computed from a batch it was
 * just served (the reference model's log-probs, the reward, ...), which is how readiness cascades
 * from generation through the inference states to the actor update (Fig. 1, Fig. 2): the samples
 * are the ones the get returned, and their number is read from the get's result block on the
 * device when the put executes, so the host neither waits for the get nor learns its size.
 *   batch        the td_get_out of that get (host struct, device pointers): indices, cu_prompt,
 *                cu_response and result are used and must stay valid until the put has executed;
 *                the put must be ordered behind the get (same stream, or an event).
 *   max_samples  upper bound of the batch size (the value given to the get).
 *   items        host array; column `column` takes row i of the batch from d_data (device) at
 *                element cu_<class>[i], i.e. rows packed in batch order exactly as a packed get
 *                lays them out; a TD_SCALAR column takes element i.  data_elems bounds what is
 *                read.
 * Everything else is td_put_many's: rows are placed and checked the same way, and the same
 * conditions are counted. */
typedef struct {
    uint32_t column, reserved;
    const void *d_data;
    uint64_t data_elems;
} td_back_item;
int td_put_back(td_dock *dock, const td_get_out *batch, uint32_t max_samples, const td_back_item *items,
                uint32_t n_items, void *stream);

/* The write-backs of several worker states in one call (three kernel launches for up to eight
 * of them): request r sends column `column` back for the batch `batch` it names, exactly as
 * td_put_back(dock, batch, max_samples, {column, d_data, data_elems}, 1, stream) would; the
 * requests are stored in array order.  Together with td_get_many this serves one poll of every
 * worker state with five or six launches, whatever their number. */
typedef struct {
    const td_get_out *batch;
    uint32_t max_samples, column;
    const void *d_data;
    uint64_t data_elems;
} td_back_req;
int td_put_back_many(td_dock *dock, const td_back_req *reqs, uint32_t n_reqs, void *stream);

/* Many gets served by one call.  Each worker state has its own controller and a step serves
 * several of them, each in several micro-batches; a plan fixes the list of requests (consumer,
 * max_samples, output buffers) once and td_get_many then serves all of them with three kernel
 * launches (two when the dock has at most 1024 prompts and every consumer one request).  Requests that name the same consumer are served in array order: the result is the
 * one td_get would give when called on each request in turn, except that a group cut off by
 * TD_ERR_OUT_TRUNCATED is not offered to the later requests of the same call.
 *   td_plan_bytes   device bytes a plan of n_req requests needs (request table + scan scratch).
 *   td_plan_create  checks the requests (host array; out.scratch is not used), uploads them into
 *                   d_plan (device, 256-byte aligned, caller-owned, must outlive the plan) on
 *                   `stream`.  n_req * n_columns must not exceed 4096, and the requests' output
 *                   room together must stay below 256 GiB (TD_EINVAL).
 *   td_get_many     enqueues the gets.  A plan must not be in flight twice at the same time;
 *                   reusing it on one stream, call after call, is the intended use. */
typedef struct {
    uint32_t consumer, max_samples;
    td_get_out out;
} td_get_req;
typedef struct td_plan td_plan;
size_t td_plan_bytes(const td_dock *dock, uint32_t n_req);
int td_plan_create(td_dock *dock, const td_get_req *reqs, uint32_t n_req, void *d_plan,
                   size_t plan_bytes, void *stream, td_plan **out);
int td_plan_destroy(td_plan *plan);
int td_get_many(td_dock *dock, td_plan *plan, void *stream);

/* One buffer serves one RL iteration: forget every table, bitmap and counter; payload bytes
 * and capacities stay. */
int td_reset(td_dock *dock, void *stream);

/* Synchronises `stream`, then copies counters and the error word to *host_out. */
int td_status(td_dock *dock, td_stats *host_out, void *stream);

/* Device address and size of an internal table, for inspection by tests and tools.
 *   which: 0 status u32[n] | 1 len i32[n] (index = class) | 2 off i64[n] (index = class)
 *          3 cursor u64[S] (index = class) | 4 claim bits (index = consumer)
 *          5 consumed bits (index = consumer) | 6 arena or scalar store (index = column) */
int td_debug_table(const td_dock *dock, int which, uint32_t index, void **d_ptr, size_t *bytes);

/* Self-check of the dock's bookkeeping, for tests and for tracking down a misbehaving caller:
 * synchronises `stream`, copies the tables to the host and tests what must hold between any two
 * calls: a stored column implies a reserved row; the rows of a warehouse (the split of the buffer
 * along the batch, "Distributed Transfer Dock Strategy") start on row boundaries, do not overlap
 * and end below the shard's cursor, which stays within the capacity; status words carry no
 * unknown bits; a sample marked served belongs to a claimed group and had every column its
 * consumer needs; the per-column and per-consumer counters equal what the tables say.
 * (While a get is in flight on another stream the claim of a group may be ahead of its served
 * marks; that is not reported.)  violations = 0 means all hold; first_sample names a sample,
 * shard, column or consumer of the first violation found. */
enum {
    TD_BAD_STORED_WITHOUT_ROW = 1u << 0,
    TD_BAD_ROW_PLACEMENT      = 1u << 1,
    TD_BAD_ROW_OVERLAP        = 1u << 2,
    TD_BAD_STATUS_BITS        = 1u << 3,
    TD_BAD_SERVED_UNCLAIMED   = 1u << 4,
    TD_BAD_SERVED_NOT_READY   = 1u << 5,
    TD_BAD_COUNTERS           = 1u << 6
};
typedef struct {
    uint32_t violations, reserved;
    uint64_t first_sample;
    uint64_t stored[32];             /* per column: samples whose status carries its bit */
    uint64_t served[32];             /* per consumer: samples marked served */
    uint64_t arena_elems_used[3];    /* by length class: elements taken by rows, padding included */
} td_validate_report;
int td_debug_validate(td_dock *dock, void *stream, td_validate_report *report);

/* Test hook for the bounded wait of the readiness scan (workflow step 1): a scan tile waits at
 * most poll_limit polls for the tiles ahead of it (0 restores the default, about 2^20), and the
 * tile that draws number skip_tile withholds its descriptor (UINT32_MAX: none), so that the
 * waits of the tiles behind it run out.  Such a get serves nothing, reports
 * TD_ERR_LOOKBACK_TIMEOUT in its result and in the error word, counts n_lookback_timeouts, and
 * hands every claim it made back.  Only this wait is affected; waits on staged copies keep
 * their own limit.  Applies to gets enqueued after the call; not to be called while other host
 * threads are using the dock. */
int td_debug_lookback(td_dock *dock, uint32_t poll_limit, uint32_t skip_tile);

/* Kernels this dock has launched since td_create. */
uint64_t td_launch_count(const td_dock *dock);

/* Per-launch timing of the two copy kernels, the ones that move Eq. 1's payload terms:
 * which = 0 the put scatter, 1 the get gather.  While enabled, each of their launches is
 * bracketed by a pair of CUDA events on the launching stream (host objects; no device memory).
 * td_kernel_timing(dock, enable) clears what was collected and switches collection on or off;
 * td_kernel_timing_read waits for the recorded launches and returns their count and summed
 * device time in milliseconds. */
int td_kernel_timing(td_dock *dock, int enable);
int td_kernel_timing_read(td_dock *dock, int which, uint64_t *launches, double *total_ms);

/* Host-buffer variants: the same workflow steps for a worker whose tensors live in host memory,
 * with the transfers across the bus part of the call (the paper's workers exchange samples
 * between nodes; here the hop is host <-> device).
 * td_put_host: h_indices / h_cu / h_data are HOST arrays (pinned memory makes the copies
 * asynchronous); they are copied into d_stage (device, 256-byte aligned, at least
 * td_put_host_stage_bytes() bytes, not reused until the put has executed) and put from there.
 * td_get_host: runs td_get into the device buffers of dev_out, then copies exactly the valid
 * part of every buffer to the matching HOST pointer of host_out (NULL = skip; host_out->result
 * and host_out->indices are required; col_capacity_elems bounds the host buffers).  It
 * synchronises the stream twice and returns with host_out filled. */
size_t td_put_host_stage_bytes(const td_dock *dock, uint32_t column, uint32_t k, uint64_t data_elems);
int td_put_host(td_dock *dock, uint32_t column, const int32_t *h_indices, uint32_t k,
                const int32_t *h_cu, const void *h_data, uint64_t data_elems,
                void *d_stage, size_t stage_bytes, void *stream);
int td_get_host(td_dock *dock, uint32_t consumer, uint32_t max_samples, const td_get_out *dev_out,
                const td_get_out *host_out, void *stream);
/* The batched calls with host buffers.
 * td_put_many_host: td_put_many whose items' three pointers (named d_* in td_put_item) are HOST
 * arrays here; they are copied, item after item, into d_stage (device, 256-byte aligned, at
 * least the sum of td_put_host_stage_bytes() over the items, not reused until the put has
 * executed) and put from there with one td_put_many; an index or cu array that several items
 * of the call name (same host pointer, same k) is brought over once.
 * td_get_many_host: td_get_many on `plan`, then the valid part of every request's buffers is
 * copied to the matching HOST pointers of host_outs[r] (one entry per request of the plan, in
 * plan order; result and indices required, NULL elsewhere = skip).  All result blocks are
 * fetched behind one synchronisation, all payload behind a second one: two per call however many
 * requests the plan holds, where td_get_host takes two per request.  d_stage (device, 16-byte
 * aligned, td_get_many_host_stage_bytes(plan) bytes, private to the call) is optional: with it
 * the get writes every request's result block, indices, cu_seqlens and advantages a second time,
 * side by side, and one transfer brings them all to the host (the first such call on a plan
 * allocates a pinned host buffer of that size, freed by td_plan_destroy); NULL: one transfer per
 * array and request. */
int td_put_many_host(td_dock *dock, const td_put_item *h_items, uint32_t n_items, void *d_stage,
                     size_t stage_bytes, void *stream);
size_t td_get_many_host_stage_bytes(const td_plan *plan);
int td_get_many_host(td_dock *dock, td_plan *plan, const td_get_out *host_outs, uint32_t n_req, void *d_stage,
                     size_t stage_bytes, void *stream);

/* The communication-volume model of "Distributed Transfer Dock Strategy", in bytes, for sizing a
 * dock or a link (host arithmetic only; no device is touched):
 *   cv        Eq. 1: what one actor-update request takes out of a centralized replay buffer,
 *             G*N*B*(PL + n*SL + M);
 *   tcv       Eq. 2: the total over the last three steps of the replay-buffer workflow,
 *             G*N*B*(2*PL + 3*n*SL + 8*M)                         (Table 1 prints it in GB = 2^30 B);
 *   tcv_dock  Eq. 4: the share of one of S warehouses when C controllers hold the metadata,
 *             G*N*B*(2*PL + 3*n*SL + 8*(C+1)*M) / S               (a double: S need not divide).
 * G prompts, N responses per prompt, PL / SL maximum prompt / response length, n response-length
 * items and M scalars per sample, B bytes per element.  Any out pointer may be NULL.
 * TD_EINVAL: NULL model, S = 0, or a product that does not fit 64 bits. */
typedef struct {
    uint64_t G, N, PL, n, SL, M, B;
    uint64_t C, S;                     /* Eq. 4 only */
} td_model;
int td_model_bytes(const td_model *m, uint64_t *cv, uint64_t *tcv, double *tcv_dock);

const char *td_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* TD_H */
