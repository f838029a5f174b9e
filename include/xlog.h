/* xlog.h -- C ABI of the B200 tagged-Datalog fixpoint engine.
 *
 * The library evaluates Datalog-style rules bottom-up over GPU-resident relations
 * whose tuples carry an fp32 tag from a semiring, with the semi-naive loop of the
 * paper's Algorithm 1 ("Semi-naive evaluation on GPU"): join the delta with the
 * full relation, project the head, combine tags per head key, remove what the full
 * relation already holds (keeping strict tag improvements) and merge, until
 * nothing changes.  Relational steps follow the paper's kernel table ("Relational
 * kernels": join, sort, groupby, dedup, set_ops, scan, pack); head aggregates are
 * those of "Aggregations and constraints" (count, sum, min, max, logsumexp).
 *
 * Conventions
 *   - every function returns an xlog_status, never throws, never aborts; outputs
 *     are untouched on failure; xlog_last_error() gives a message;
 *   - pointers are HOST pointers unless a parameter says xlog_memspace or "device";
 *   - the caller owns every buffer it passes in (arena, inputs, outputs); the
 *     context owns what it carves from the arena; nothing is freed across the
 *     boundary; the library calls no cudaMalloc for relation data;
 *   - all device work is issued on the stream given at context creation and every
 *     entry point is stream-synchronous on return;
 *   - a context is not thread-safe; there is no process-wide state
 *     (Section "Crate architecture": no runtime singleton), except the per-device
 *     scratch array of xlog_reduce_by_key_static (see there).
 *   - keys are int32 and must be >= 0 (dense ids, Section "Reversible symbols").
 */
#ifndef XLOG_H
#define XLOG_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define XLOG_MAX_ARITY 4
#define XLOG_MAX_ATOMS 4
#define XLOG_MAX_VARS  8

/* Typed outcomes (Section "GPU residency model": RESOURCE_EXHAUSTED for bytes,
 * CAPACITY_EXCEEDED for counts, CONVERGENCE_FAILURE for the iteration limit). */
typedef enum {
  XLOG_OK = 0,
  XLOG_ERR_INVALID_ARGUMENT = 1,
  XLOG_ERR_INVALID_VALUE = 2,        /* NaN tag, tag equal to the semiring zero, negative key */
  XLOG_ERR_UNSUPPORTED = 3,          /* plan shape; a non-linear rule under logsumexp / sum inside a recursive component */
  XLOG_ERR_RESOURCE_EXHAUSTED = 4,   /* arena bytes */
  XLOG_ERR_CAPACITY_EXCEEDED = 5,    /* key bits > 64, count > INT32_MAX, head value outside [0, 2^31) */
  XLOG_ERR_CONVERGENCE_FAILURE = 6,  /* iteration cap reached */
  XLOG_ERR_BUFFER_TOO_SMALL = 7,
  XLOG_ERR_INVALID_STATE = 8,        /* derived relations poisoned by an earlier failure */
  XLOG_ERR_CUDA = 9,
  XLOG_ERR_INTERNAL = 10
} xlog_status;

/* (oplus, otimes, zero, one): MAXPLUS (max,+,-inf,0)  MINPLUS (min,+,+inf,0)
 * LOGSUMEXP (logaddexp,+,-inf,0)  SUMPROD (+,*,0,1). */
typedef enum { XLOG_SR_MAXPLUS = 0, XLOG_SR_MINPLUS = 1, XLOG_SR_LOGSUMEXP = 2, XLOG_SR_SUMPROD = 3 } xlog_semiring;
typedef enum { XLOG_MEM_HOST = 0, XLOG_MEM_DEVICE = 1 } xlog_memspace;

typedef struct xlog_ctx xlog_ctx;
typedef int32_t xlog_rel;      /* relation handle, valid for the context that made it */
typedef int32_t xlog_rule;     /* rule handle */

typedef struct {
  uint32_t struct_size;            /* sizeof(xlog_config) */
  int32_t  device;                 /* CUDA device ordinal the arena lives on */
  void*    stream;                 /* cudaStream_t, may be NULL (default stream) */
  void*    arena;                  /* DEVICE memory, >= 256-byte aligned, owned by the caller, must outlive the ctx */
  uint64_t arena_bytes;
  int64_t  max_iterations;         /* per recursive component; <= 0 means 2^20 */
  uint64_t candidate_chunk_bytes;  /* upper bound on one batch of join candidates; 0 = bounded by the arena only */
  uint32_t flags;                  /* XLOG_FLAG_* */
} xlog_config;

#define XLOG_FLAG_CHECK_INVARIANTS 1u  /* after every load/merge verify keys strictly increase (slow, for tests) */
#define XLOG_FLAG_PROFILE          2u  /* CUDA events around every kernel launch; read with xlog_profile_read */
#define XLOG_FLAG_NO_TAG_MIRROR    4u  /* evaluate every recursive component by sort -> reduce-by-key -> merge */
#define XLOG_FLAG_NO_RESIDENT_LOOP 8u  /* the host drives every round of a tag-mirror fixpoint (one control read per round) */
#define XLOG_FLAG_FORCE_WCOJ      32u  /* materialised triangle joins: always the multiway (worst-case-optimal) plan */
#define XLOG_FLAG_FORCE_CHAIN     64u  /* ... always the binary-join chain (fails with RESOURCE_EXHAUSTED if its intermediate does not fit) */
#define XLOG_FLAG_NO_GROUPED_JOIN 128u  /* tag mirror: always the row-wise join, never the grouped one (see csrc/group_join.cuh) */
#define XLOG_FLAG_NO_BITMAP_JOIN  256u  /* tag mirror, grouped join: always from a delta row list, never straight from the changed bitmap (see csrc/bitmap_join.cuh) */
#define XLOG_FLAG_NO_DENSE_DOUBLING 512u /* tag mirror: the path-doubling rule h(x,z) :- h(x,y), h(y,z) goes through the sorting route, not the dense rounds */
#define XLOG_FLAG_NO_TRIANGLE_BITMAP 1024u /* fused triangle aggregate: always search the longer list, never mark in(x) in a shared-memory bitmap (see csrc/triangle.cuh) */
#define XLOG_FLAG_NO_ROW_FIXPOINT 2048u /* tag mirror, h(a,c) :- h(a,b), r(b,c): never run the rounds of each a on their own in shared memory (see csrc/row_fixpoint.cuh) */
#define XLOG_FLAG_NO_GRAPH        16u  /* resident rounds are launched one by one instead of as one graph with a WHILE node */

/* Evaluation routes of a recursive component (Algorithm 1).  All of them derive the same relation,
 * bit for bit, and the same receipt counters (unique_candidates excepted, see xlog_receipt).
 *  - Sorting route: join -> sort -> reduce-by-key -> merge-path difference, as in the paper's kernel table.
 *  - Tag mirror (default where it applies: one MAXPLUS/MINPLUS head relation, every rule with at most one
 *    atom over it and that atom scanned, packed key <= 30 bits, table fits the arena): the relation is a
 *    direct-addressed table of one tag per possible key; candidates are applied with one atomic max/min.
 *    Above 2^24 possible keys a rule of the shape h(a, c) :- h(a, b), r(b, c) is joined "grouped": the mirror is
 *    indexed with the probed column as the major part, the delta comes out grouped by b, and the delta rows of one b
 *    share the read of r's run of b and a line of the table (XLOG_FLAG_NO_GROUPED_JOIN switches this off).  With at
 *    least 32 (and at most 1024) possible values of a and one such rule, the rounds are driven by the changed bitmap itself:
 *    one kernel turns the bitmap into work items and a list of the changed keys' (tag, a) pairs grouped by b, one joins
 *    (XLOG_FLAG_NO_BITMAP_JOIN switches this off); the pair list holds 8 bytes per possible key.
 *    One rule shape with two atoms over the relation is served as well: path doubling  h(x,z) :- h(x,y), h(y,z)  as the
 *    only rule over a binary h with at most 4096 values in its second column.  The mirror is then a matrix; a round copies
 *    it (the state both delta variants read) and one thread block per row applies every candidate of both variants in
 *    shared memory (csrc/dense_closure.cuh; XLOG_FLAG_NO_DENSE_DOUBLING sends the rule through the sorting route).
 *  - Row-local fixpoint (tag mirror, one rule of the shape h(a, c) :- h(a, b), r(b, c) over h, at most 8192 possible values
 *    of c): the rule never changes a, so the rounds of each a are independent; after the seed round one launch runs every
 *    a's rounds to the end, a thread block per a with that a's slots in shared memory; several mutually recursive heads
 *    whose rules all read h_i(a, c) :- h_j(a, b), r(b, c) and that share one key layout are handled alike (csrc/row_fixpoint.cuh;
 *    XLOG_FLAG_NO_ROW_FIXPOINT, and the flags that select the routes below, switch it off).
 *  - Resident rounds (tag mirror with <= 2^24 possible keys): the delta rounds run as one CUDA graph with a
 *    conditional WHILE node and fixed-capacity buffers (Section "GPU-Native Symbolic Substrate": resident
 *    conditional graph, no host reads inside the loop).  The buffers (about 36 bytes per possible key
 *    plus 12 MB) and the instantiated graph stay allocated in the arena from the first such xlog_fixpoint
 *    until the context is destroyed or the relation's key layout changes.  The first call also
 *    creates a private stream that records the graph; nothing else ever runs on it. */

/* ---- context --------------------------------------------------------------- */
xlog_status xlog_ctx_create(const xlog_config* cfg, xlog_ctx** out);
xlog_status xlog_ctx_destroy(xlog_ctx* ctx);          /* frees host state and the pinned control block only */
const char* xlog_last_error(const xlog_ctx* ctx);     /* owned by ctx, valid until the next call on it */

/* ---- relations (Section "Type system": typed columnar predicates) ------------ */
/* arity 1..XLOG_MAX_ARITY.  The packed key of a row (all columns, bit widths taken
 * from the column maxima) must fit 64 bits, else CAPACITY_EXCEEDED at load/fixpoint. */
xlog_status xlog_relation_create(xlog_ctx* ctx, int32_t arity, xlog_semiring sr, const char* name, xlog_rel* out);

/* Replace the relation's facts by n rows given column-major: cols[c][i], tags[i]
 * (tags == NULL loads the semiring one).  COPIES the data (space says where cols/tags
 * live), sorts lexicographically, combines rows with equal keys by oplus, canonicalises
 * -0.0 to +0.0, stores int32 columns + fp32 tag column-major.  Rejects negative keys,
 * NaN tags and (except SUMPROD) tags equal to the semiring zero with INVALID_VALUE.
 * Any load drops all derived tuples of the context (as xlog_ctx_reset_idb). */
xlog_status xlog_relation_load(xlog_ctx* ctx, xlog_rel rel, const int32_t* const* cols, const float* tags,
                               int64_t n, xlog_memspace space);

xlog_status xlog_relation_size(xlog_ctx* ctx, xlog_rel rel, int64_t* n);

/* Copy the relation out in ascending lexicographic key order.  cols_out[c] and
 * tags_out each hold `capacity` elements in `space`; BUFFER_TOO_SMALL if n > capacity. */
xlog_status xlog_relation_read(xlog_ctx* ctx, xlog_rel rel, int32_t* const* cols_out, float* tags_out,
                               int64_t capacity, int64_t* n_out, xlog_memspace space);

/* Zero-copy DEVICE pointers to the stored columns (Section "Zero-copy
 * interoperability"); borrowed, valid until the relation next changes. */
xlog_status xlog_relation_view(xlog_ctx* ctx, xlog_rel rel, const int32_t** cols /*[arity]*/, const float** tags, int64_t* n);

/* ---- rules: a compiled conjunctive plan ---------------------------------------
 * Each atom argument is a constant or an affine pattern  column == mul*var + add
 * (mul > 0; rows that do not divide evenly do not match).  Equal var ids are join
 * keys.  Head column c is  c0 + sum_v coef[v]*var_v  evaluated in int64; a value
 * outside [0, 2^31) fails the fixpoint with CAPACITY_EXCEEDED.  The head tag is
 * the otimes-product of the atom tags in atom order, combined per head key with the
 * HEAD relation's oplus.  emit_count_column appends the number of bindings of the
 * group as a trailing int32 head column (the paper's count is a head column:
 * Listing 7), so the head relation's arity is n_head_cols + 1.
 * Supported shapes: 1 atom; 2 atoms joined on one variable, the second side looked
 * up through a sorted index on that column, its other columns plain variables;
 * the 3-atom triangle join, either aggregated per x over one binary relation,
 * h(x[, count]) :- e(x,y), e(y,z), e(z,x)  (fused intersect-and-aggregate, nothing
 * materialised), or materialised over up to three binary relations,
 * h(x,y,z) :- r(x,y), s(y,z), t(z,x)  (rows born sorted).  The materialised form has two
 * plans (Sections "Worst-case-optimal joins", "WCOJ vs. the binary-join plan"): the
 * multiway join (count -> scan -> write per row of r, intersecting s's out-list of y with
 * t's in-list of x) and the binary-join chain (all two-paths of r and s, then a probe of
 * t).  A skew test chooses per evaluation: the chain when the two-paths, counted exactly,
 * number at most four per input row of the largest relation and fit the arena, the
 * multiway join otherwise; XLOG_FLAG_FORCE_WCOJ / XLOG_FLAG_FORCE_CHAIN override it and
 * xlog_receipt.triangle_plan reports the choice.  Both plans produce identical rows.
 * The four-cycle join  h(x,y,z,w) :- r(x,y), s(y,z), t(z,w), u(w,x)  (same sections: coverage
 * spans the triangle and 4-cycles) over up to four binary relations, head columns exactly
 * (x,y,z,w): the two-paths of r and s, then either the multiway step (per two-path the
 * intersection of t's out-list of z with u's in-list of x, count -> scan -> write) or the rest of
 * the binary-join chain (every three-path of r, s, t written out, then a probe of u).  The same
 * skew test chooses, on the exact three-path count; the same flags override it and
 * xlog_receipt.triangle_plan reports the choice; both plans produce identical rows, sorted.  It
 * must be the only rule of its head, outside recursion; RESOURCE_EXHAUSTED if the two-paths do
 * not fit the arena.
 * Negation (Sections "Aggregations and constraints", "Completeness over finite domains":
 * explicit stratified negation-as-failure): a rule of one positive atom followed by one
 * negated atom,  h(..) :- a(..), not b(..).  The negated atom holds iff no row of b matches;
 * its first column, or its first two, must be fixed by constants / variables of the positive
 * atom, the remaining columns must be variables that occur nowhere else (wildcards); it adds
 * nothing to the tag; b must belong to a lower stratum.  Anything
 * else: UNSUPPORTED.  Which atoms are recursive is derived from the strongly
 * connected components of the relation dependency graph; a rule may have one or two
 * recursive atoms (p(x,z) :- p(x,y), p(y,z) is evaluated with one delta variant per
 * occurrence, Section "Semi-naive evaluation on GPU"), and a component may hold
 * several mutually recursive relations (MAXPLUS / MINPLUS heads whose rules each read one
 * relation of the component are evaluated over one tag mirror per head, see below; other
 * shapes by sort, reduce-by-key and merge).
 * Tags inside recursion: a component of MAXPLUS / MINPLUS relations runs Algorithm 1 with tag
 * improvement (a tuple re-enters the delta when its tag strictly improves).  A component of
 * LOGSUMEXP or SUMPROD relations (Section "Aggregations and constraints" rejects aggregation
 * inside a recursive component; this is the extension to acyclic derivations) must have at most
 * one recursive atom per rule; the tag of a tuple is then the oplus over ALL its derivations
 * (path counts, sums of path products), evaluated with deltas that carry tag differences, and
 * recomputed from the loaded facts on every xlog_fixpoint.  If the derivations are cyclic the
 * rounds never end: CONVERGENCE_FAILURE at max_iterations.  Mixed components: UNSUPPORTED. */
typedef enum { XLOG_ARG_CONST = 0, XLOG_ARG_VAR = 1 } xlog_arg_kind;
typedef struct { int32_t kind; int32_t var; int32_t mul; int32_t add; /* CONST: add is the value */ } xlog_arg;
typedef struct { xlog_rel rel; xlog_arg args[XLOG_MAX_ARITY]; int32_t negated; /* 1: negation as failure, see below */ } xlog_atom;
typedef struct { int64_t c0; int32_t coef[XLOG_MAX_VARS]; } xlog_expr;
typedef struct {
  uint32_t  struct_size;           /* sizeof(xlog_plan) */
  xlog_rel  head_rel;
  int32_t   n_head_cols;
  xlog_expr head[XLOG_MAX_ARITY];
  int32_t   n_atoms;
  xlog_atom atoms[XLOG_MAX_ATOMS];
  int32_t   emit_count_column;
} xlog_plan;

xlog_status xlog_rule_add(xlog_ctx* ctx, const xlog_plan* plan, xlog_rule* out);   /* validates and copies */

/* ---- evaluation ------------------------------------------------------------- */
/* Terminal receipt: status, counters and timing, never tuple data (Section
 * "GPU-Native Symbolic Substrate"). */
typedef struct {
  uint32_t struct_size;            /* sizeof(xlog_receipt), set by the caller */
  int32_t  status;
  int64_t  strata;                 /* components evaluated */
  int64_t  iterations;             /* join rounds over all components, seed rounds included */
  int64_t  derived_tuples;         /* sum over rule heads of rows - loaded facts */
  int64_t  candidates;             /* join outputs before aggregation */
  int64_t  unique_candidates;      /* after reduce-by-key; -1 if a component was evaluated through a tag mirror,
                                      which never forms the list of distinct candidate keys */
  int64_t  new_tuples;
  int64_t  improved_tags;
  int64_t  h2d_bytes, d2h_bytes;   /* control traffic of this call (counters only) */
  int64_t  kernel_launches;
  int64_t  peak_arena_bytes;
  double   device_ms;              /* CUDA-event time of the whole call on the ctx stream */
  int32_t  triangle_plan;          /* XLOG_PLAN_*: how the last materialised triangle or four-cycle join of this call was evaluated */
  int32_t  index_builds;           /* join indices (offsets over a column, permuted sorted copies) built during this call: indices
                                      of relations that did not change since an earlier call are reused, not rebuilt
                                      (Sections "Runtime optimization", "Index reuse and the chain scorer") */
} xlog_receipt;
#define XLOG_PLAN_NONE  0
#define XLOG_PLAN_WCOJ  1          /* multiway join: per row of the first atom, intersect two sorted lists */
#define XLOG_PLAN_CHAIN 2          /* binary-join chain: materialise the two-paths, then probe the third atom */

/* Evaluate all rules to the least fixpoint, strata in dependency order
 * (Algorithm 1; non-recursive components evaluate each rule once).  On failure
 * the derived relations are poisoned: every later call that needs them returns
 * INVALID_STATE until xlog_ctx_reset_idb (counters of a failed run are not a
 * result: Section "Current limitations").  receipt may be NULL. */
xlog_status xlog_fixpoint(xlog_ctx* ctx, xlog_receipt* receipt);

/* Drop all derived tuples; loaded facts and their join indices stay. */
xlog_status xlog_ctx_reset_idb(xlog_ctx* ctx);

/* Gradient of a non-recursive LOGSUMEXP (or SUMPROD) rule after a successful
 * fixpoint (the quantity the paper obtains by circuit backward, Section
 * "End-to-end training").  grad_head: DEVICE, one float per head row in stored
 * order.  grad_atoms[j]: DEVICE, one float per row of atom j's relation in stored
 * order; each distinct buffer is zero-filled first, then
 *   LOGSUMEXP:  grad_j[row] += g[h] * exp(sum_i tag_i - out[h])
 *   SUMPROD:    grad_j[row] += g[h] * prod_{i != j} tag_i
 * Passing the same pointer for two atoms of one relation yields the sum.  A pointer
 * whose relation holds no rows may be NULL; otherwise NULL is INVALID_ARGUMENT. */
xlog_status xlog_rule_backward(xlog_ctx* ctx, xlog_rule rule, const float* grad_head, float* const* grad_atoms);

/* ---- the sort on its own (paper kernel table: `sort`) ---------------------------------
 * Stable ascending sort of n (key, 4-byte payload) pairs by the low key_bits bits of the key.
 * keys / payload: DEVICE, sorted in place; key_bytes is 4 or 8; n < 2^30.  Scratch (a second
 * buffer pair and the pass bookkeeping) comes from the context's arena: RESOURCE_EXHAUSTED if
 * it does not fit.  Used by load, by index builds and once per round by the fixpoint. */
xlog_status xlog_sort_pairs(xlog_ctx* ctx, void* keys, void* payload, int64_t n, int32_t key_bytes, int32_t key_bits);

/* ---- per-kernel statistics (Section "Semi-naive evaluation on GPU": the profiler records
 * per-operator timing and row counts) ------------------------------------------------
 * With XLOG_FLAG_PROFILE every kernel launch is bracketed by CUDA events on the context's
 * stream.  xlog_profile_read waits for the stream, then writes one entry per kernel
 * (accumulated since creation or the last reset): launches, summed device time, and the
 * algorithmic bytes the launch sites declared (0 for helper kernels).  out may be NULL to
 * query the count; at most `capacity` entries are written. */
typedef struct {
  char    name[48];
  int64_t launches;
  double  device_ms;
  int64_t algorithmic_bytes;
} xlog_kernel_stat;
xlog_status xlog_profile_read(xlog_ctx* ctx, xlog_kernel_stat* out, int32_t capacity, int32_t* n_out);
xlog_status xlog_profile_reset(xlog_ctx* ctx);

/* ---- a plain copy kernel, for measuring (The paper has no counterpart.) ----------------------------------------------
 * Copies `bytes` (a multiple of 16; both pointers DEVICE, 16-byte aligned, not overlapping) from src to dst `repeats`
 * times with the library's own grid-stride 16-byte-vector kernel, on `stream`, without waiting.  The benchmark times it
 * on a buffer pair smaller than L2 to obtain the L2 bandwidth that cache-resident kernels (the sorted-list intersections
 * of the triangle and four-cycle joins) are reported against, and on a large pair as a cross-check of the HBM figure. */
xlog_status xlog_device_copy(void* stream, void* dst, const void* src, uint64_t bytes, int32_t repeats);
/* The read-only counterpart: reads `bytes` (a multiple of 16; src DEVICE, 16-byte aligned) `repeats` times, eight 16-byte loads
 * per thread in flight, and writes nothing (`sink`: 4 writable DEVICE bytes, 4-byte aligned, that keep the loads alive; they
 * are stored to only if the XOR of a thread's words takes one particular value).  The join kernels that are held against the
 * L2 rate mostly read, so the benchmark reports them against the higher of the two figures.  Same error behaviour as above:
 * XLOG_ERR_INVALID_ARGUMENT for a null or misaligned pointer, a size that is not a multiple of 16 or repeats < 1. */
xlog_status xlog_device_read(void* stream, const void* src, uint64_t bytes, int32_t repeats, void* sink);
/* Random reads: at least `reads` 4-byte loads (rounded up to a multiple of 8 per thread of a fixed grid) at hashed word
 * offsets of the `bytes`-byte table at src (DEVICE, 4-byte aligned, 4 <= bytes <= 2^34, a multiple of 4), eight per thread
 * in flight; nothing is written (`sink` as above).  Each load touches one 32-byte sector: the rate is what the row-wise
 * tag-mirror join (one table slot per candidate) is held against. */
xlog_status xlog_device_gather(void* stream, const void* src, uint64_t bytes, uint64_t reads, void* sink);

/* ---- failure-path hooks (tests only) -----------------------------------------------------
 * Two kernels wait for other thread blocks of their own launch: the sort pass and the resident count + scan look back
 * through per-tile status words.  A tile only waits for tiles that already run, and every wait gives up after a number
 * of polls, raises the device error flag, writes nothing more and lets the call fail with XLOG_ERR_INTERNAL (typed,
 * fail-closed outcomes: Section "GPU residency model").  The default limit (2^22 polls) is never reached in a healthy run.
 * xlog_debug_set_poll_limit lowers it for this context; xlog_debug_sort_pass_without_first_tile runs one 8-bit sort pass
 * (keys / payload -> out_keys / out_payload, all DEVICE, n rows, at least two tiles of 4096) in which the first tile is
 * deliberately not launched, so that every other tile's wait runs out: the call returns XLOG_ERR_INTERNAL, the outputs
 * stay as they were, and the context remains usable. */
xlog_status xlog_debug_set_poll_limit(xlog_ctx* ctx, uint32_t polls);
xlog_status xlog_debug_sort_pass_without_first_tile(xlog_ctx* ctx, const void* keys, const void* payload, void* out_keys, void* out_payload,
                                                    int64_t n, int32_t key_bytes);

/* ---- reduce-by-key that allocates nothing --------------------------------------------
 * (The paper has no counterpart for this entry point.)
 *
 * For callers that cannot allocate device memory at call time: a serving loop whose memory
 * was all handed out at start-up, a process whose device pool belongs to another component,
 * or a stream that must not see the implicit synchronisation an allocation can cause.  It
 * needs no context and no arena: the scratch of the segmented reduction lives in a fixed
 * device array inside the library (about 164 KB, held by every GPU that loads the library
 * until the process exits), which bounds the input at XLOG_STATIC_REDUCE_MAX_ROWS rows.
 *
 * Input: n rows with keys ascending (equal keys adjacent, keys >= 0) and their tags, both
 * DEVICE pointers.  Output: one row per distinct key with the oplus of its tags under `sr`
 * (same arithmetic as the engine's group-by), written to out_keys / out_tags (DEVICE, room
 * for n rows; an output that overlaps an input or the other output is rejected with
 * INVALID_ARGUMENT); *n_out (HOST) receives the number of groups.
 * errbuf (HOST, optional) receives a message on failure.
 *
 * Returns CAPACITY_EXCEEDED, touching nothing, when n > XLOG_STATIC_REDUCE_MAX_ROWS.
 * Calls no cudaMalloc / cudaFree or other allocating routine.  Runs on `stream` of the
 * CURRENT device and waits for it before returning.  The first call on each device also
 * looks up the array's device address (once per device); make that first call before
 * starting any stream capture.  All calls on a device share the one array, which keeps
 * whatever the last call left there: each call overwrites every slot before reading it, but
 * two calls whose kernels overlap on the GPU (different streams or threads) race. */
#define XLOG_STATIC_REDUCE_MAX_ROWS (1 << 24)
xlog_status xlog_reduce_by_key_static(void* stream, xlog_semiring sr, const int32_t* keys, const float* tags, int64_t n,
                                      int32_t* out_keys, float* out_tags, int64_t* n_out, char* errbuf, size_t errbuf_len);

#ifdef __cplusplus
}
#endif
#endif /* XLOG_H */
