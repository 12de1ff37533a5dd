/*
 * CPU oracle for the transfer dock's put/get sample flow.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, single-threaded statement of
 * what the dock computes; it exists so that the CUDA library can be checked
 * against something written independently of it.  Nothing in the product path
 * may call it: only the tests, the smoke check and the benchmark's CPU-baseline
 * leg do.  It shares no source, header, table or helper with the CUDA library.
 *
 * What follows the paper ("Distributed Transfer Dock Strategy", Fig. 4, Eq. 4):
 *   - warehouses split the buffer along the global batch, each sample keeps its
 *     own index                      -> shard_of(), per-shard arenas;
 *   - a controller per worker state records which samples it may still serve
 *                                     -> per-consumer claim / consumed bitmaps;
 *   - three-step workflow: metadata request, data get/put, state update that is
 *     visible to every controller    -> ora_get() select, ora_put(), status[].
 * The record schema (prompt item, several response-length items, a few scalars)
 * is the one stated under Eq. 1.  The paper fixes neither a selection order, nor
 * a storage layout, nor the advantage formula; the readings taken are stated at
 * each function.
 *
 * Pins (tests/test_oracle_*.py): identity round trip against the generator's
 * arrays, exactly-once dispatch, brute force on tiny docks against a
 * filter-sort-take definition, numpy.cumsum for cu_seqlens, numpy mean/std for
 * advantages plus closed forms (N = 2, all-equal groups), hand-computed arena
 * offsets, Eq. 1 / Eq. 2 / Eq. 4 against the printed Table 1.
 * Parity unpinned: the dispatch order under truly concurrent gets (several
 * outcomes are valid; invariants are checked instead), and the behaviour of the
 * paper's own Ray/TensorDict dock (no code or worked example is published).
 */
#ifndef TD_ORACLE_H
#define TD_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORA_I32 = 0, ORA_F32 = 1, ORA_BF16 = 2 };
enum { ORA_SCALAR = 0, ORA_PROMPT = 1, ORA_RESPONSE = 2 };
enum { ORA_PACKED = 0, ORA_PADDED = 1 };
enum { ORA_OUT_LEFT_PAD_PROMPT = 1u };             /* ora_get_out.flags */
enum { ORA_F_ADVANTAGE = 1u };

/* condition bits, OR-ed into ora_result.status and the dock's error word */
enum {
    ORA_ERR_OOB_INDEX    = 1u << 0,
    ORA_ERR_DUP_PUT      = 1u << 1,
    ORA_ERR_LEN_MISMATCH = 1u << 2,
    ORA_ERR_ARENA_FULL   = 1u << 3,
    ORA_ERR_OUT_TRUNC    = 1u << 4,
    ORA_ERR_BAD_LENGTH   = 1u << 6
};

typedef struct { int32_t dtype; int32_t cls; uint32_t pad_bits; } ora_column;
typedef struct { uint32_t need_mask, out_mask, flags; } ora_consumer;

typedef struct {
    uint32_t n_prompts, n_per_group, n_shards;      /* G, N, S; S divides G */
    uint32_t n_columns;   const ora_column *columns;
    uint32_t n_consumers; const ora_consumer *consumers;
    uint64_t prompt_elems_per_shard, response_elems_per_shard;
    uint32_t reward_column;
    float    adv_eps;
} ora_config;

typedef struct {
    uint32_t n_samples, n_groups;
    uint64_t prompt_tokens, response_tokens;
    uint32_t status;
} ora_result;

typedef struct {
    int32_t  mode;                       /* ORA_PACKED | ORA_PADDED */
    uint32_t pad_prompt_to, pad_response_to;
    uint32_t flags;                      /* ORA_OUT_LEFT_PAD_PROMPT (ORA_PADDED only): rows of prompt
                                            columns end at their width, the pad comes first */
    int32_t *indices;                    /* [max_samples] */
    int32_t *cu_prompt, *cu_response, *cu_seq;   /* [max_samples + 1] */
    void    *col[32];                    /* NULL = not wanted */
    uint64_t col_capacity_elems[32];
    float   *advantages;                 /* [max_samples] */
    ora_result *result;
    /* Fused token stream, optional (seq == NULL and seq_advantages == NULL: not wanted): sample
     * i's row of column seq_prompt_col followed by its row of column seq_response_col, at
     * element cu_seq[i] of seq; seq_advantages has the same layout in float: 0 on the prompt
     * tokens, the sample's advantage on its response tokens. */
    uint32_t seq_prompt_col, seq_response_col;
    void    *seq;
    uint64_t seq_capacity_elems;         /* bounds both */
    float   *seq_advantages;
} ora_get_out;

typedef struct {
    uint64_t put_accepted[32];
    uint64_t got_samples[32];
    uint64_t got_tokens[32];
    uint64_t n_oob, n_dup, n_len_mismatch, n_arena_full, n_truncated, n_bad_length;
    uint32_t error_word;
} ora_stats;

typedef struct ora_dock ora_dock;

ora_dock *ora_create(const ora_config *cfg);
void      ora_destroy(ora_dock *d);
void      ora_reset(ora_dock *d);
/* returns the number of accepted samples, or -1 on a bad argument */
int64_t   ora_put(ora_dock *d, uint32_t column, const int32_t *indices, uint32_t k,
                  const int32_t *cu, const void *data);
/* returns 0, or -1 on a bad argument (unknown consumer, max_samples < N, ...) */
int       ora_get(ora_dock *d, uint32_t consumer, uint32_t max_samples, const ora_get_out *out);
/* outputs for a given ascending list of sample indices, dock state untouched */
int       ora_gather(const ora_dock *d, uint32_t consumer, const int32_t *indices,
                     uint32_t count, const ora_get_out *out);
void      ora_get_stats(const ora_dock *d, ora_stats *out);

/* state inspection for parity checks */
uint32_t  ora_shard_of(const ora_dock *d, uint32_t sample);
const uint32_t *ora_status(const ora_dock *d);                 /* [n]            */
const int32_t  *ora_len(const ora_dock *d, int cls);           /* [n], -1 unset  */
const int64_t  *ora_off(const ora_dock *d, int cls);           /* [n], -1 unset  */
const uint64_t *ora_cursor(const ora_dock *d, int cls);        /* [S]            */
const uint32_t *ora_claim(const ora_dock *d, uint32_t consumer);     /* bit per group  */
const uint32_t *ora_consumed(const ora_dock *d, uint32_t consumer);  /* bit per sample */
const void     *ora_arena(const ora_dock *d, uint32_t column, uint32_t shard);
const void     *ora_scalars(const ora_dock *d, uint32_t column);

/* Communication-volume model, in GB of 1024^3 bytes: Eq. 1, Eq. 2, Eq. 4. */
double ora_cv(double G, double N, double B, double PL, double n, double SL, double M);
double ora_tcv(double G, double N, double B, double PL, double n, double SL, double M);
double ora_tcv_dock(double G, double N, double B, double PL, double n, double SL, double M,
                    double C, double S);

#ifdef __cplusplus
}
#endif
#endif
