/*
 * xg.h -- C ABI of the token-mask library (byte-level Earley, CUDA sm_100a).
 *
 * The library implements the data-parallel part of grammar-constrained decoding as described in
 * "XGrammar-2" (arXiv 2601.04426): checking every vocabulary token against a byte-level Earley
 * grammar state.  That happens in two places:
 *   - at compile time, filling the adaptive token mask cache: every (scannable grammar state,
 *     token) pair is classified accepted / rejected / uncertain (Section 3.4; appendix
 *     "XGrammar's Adaptive Token Mask cache Generation Algorithm");
 *   - at every decode step, merging the cached sets of the current scannable states with a full
 *     Earley check of the uncertain tokens (same appendix, run-time paragraph), and setting the
 *     logits of disallowed tokens to -inf (Section 2.1).
 *
 * Conventions
 *   - Every function returns an xg_status_t (0 = XG_OK, negative = error) and never throws,
 *     aborts or traps the device.  xg_last_error() returns a thread-local message for the last
 *     failing call on the calling thread.
 *   - Handles are opaque; the library creates them and the caller destroys them with the
 *     matching *_destroy.  Destroy matchers before their grammar, grammars before their
 *     tokenizer and cache pool.
 *   - "device" pointers are CUDA device memory of the current device, owned by the caller and
 *     never freed or retained past the call's stream order.  "host" pointers are ordinary memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls that take a
 *     stream only enqueue work on it unless stated otherwise.
 *   - Bitmask layout: row-major int32 words, bit j (LSB first) of word w of a row is token id
 *     32*w + j; 1 = allowed.  Bits of ids >= vocab_size are 0.
 */
#ifndef XG_H_
#define XG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t xg_status_t;
enum {
  XG_OK = 0,
  XG_ERR_INVALID_ARG = -1,
  XG_ERR_PARSE = -2,          /* grammar / schema text is malformed */
  XG_ERR_UNSUPPORTED = -3,    /* schema keyword or construct outside the supported subset */
  XG_ERR_OOM = -4,
  XG_ERR_CUDA = -5,           /* a CUDA runtime call failed, or no usable device */
  XG_ERR_CAPACITY = -6,       /* a capacity was exhausted: the matcher's history (max_sets / max_items), or an Earley
                                 set beyond even the exact slow path (2048 items per token walk) */
  XG_ERR_TOKEN_REJECTED = -7, /* xg_accept_token: the token is not allowed in this state */
  XG_ERR_TERMINATED = -8,     /* the matcher already accepted EOS */
  XG_ERR_TIMEOUT = -9,
  XG_ERR_BOUNDS = -10         /* bounds-checking build only: a kernel met an index outside its table (xg_debug_bounds_check) */
};

typedef enum { XG_EBNF = 0, XG_JSON_SCHEMA = 1, XG_TAG_DISPATCH_JSON = 2 } xg_grammar_kind_t;
typedef enum { XG_F32 = 0, XG_BF16 = 1 } xg_dtype_t;
/* how the accepted/rejected split of one cache entry is stored (the smallest of the three) */
typedef enum { XG_STORE_ACCEPT_LIST = 0, XG_STORE_REJECT_LIST = 1, XG_STORE_BITSET = 2 } xg_store_kind_t;

typedef struct xg_tokenizer xg_tokenizer_t;
typedef struct xg_cache_pool xg_cache_pool_t;
typedef struct xg_grammar xg_grammar_t;
typedef struct xg_matcher xg_matcher_t;

/* Message of the last failing call on this thread ("" if none).  Valid until the next call. */
const char* xg_last_error(void);

/* ---- bounds-checking build -----------------------------------------------------------------
 * The library can be built with -DXG_DEBUG_BOUNDS (paper_2601_04426_b200/build.py builds that variant
 * as libxg_dbg.so): its kernels range-check every index into a grammar table, the vocabulary arena, a
 * request's chart and another block's shared memory before using it.  A failed check records the first
 * violation in a device word and skips the access; nothing traps.  xg_debug_bounds_check synchronises
 * `stream`, returns XG_OK when no check has failed since the last call and XG_ERR_BOUNDS (message: which
 * table, index, limit) otherwise, and clears the word.  In the regular build the checks do not exist and
 * the call returns XG_OK.  xg_debug_bounds_enabled: 1 in the checking build, else 0. */
int32_t xg_debug_bounds_enabled(void);
xg_status_t xg_debug_bounds_check(void* stream);

/* ---- vocabulary ---------------------------------------------------------------------------
 * The token set V of the tokenizer (appendix "Formal Definitions": V is the vocabulary).
 * bytes/offsets (host): token i is bytes[offsets[i] .. offsets[i+1]).  eos_token_id = -1 for none.
 * special_ids (host, may be NULL): tokens that are never allowed.  Zero-length tokens are never
 * allowed either (EOS is decided separately).  Tokens longer than 255 bytes are refused
 * (XG_ERR_UNSUPPORTED).  The library copies everything; it stores the tokens on the device
 * sorted by their bytes (trie order) with the permutation back to ids.  Synchronous. */
xg_status_t xg_tokenizer_create(const uint8_t* bytes, const int64_t* offsets, int32_t vocab_size,
                                int32_t eos_token_id, const int32_t* special_ids, int32_t n_special,
                                void* stream, xg_tokenizer_t** out);
void xg_tokenizer_destroy(xg_tokenizer_t* tok);

/* ---- cross-grammar cache pool (Section 3.3) -----------------------------------------------
 * Cache entries are keyed by the structural hash of the rule automaton they belong to
 * (Algorithm 1; Algorithm 2 for cycles) and verified against the canonical serialisation, so
 * identical sub-structures in different grammars, or inside one grammar, are built once.
 * A pool belongs to one tokenizer and must outlive the grammars compiled with it. */
xg_status_t xg_cache_pool_create(const xg_tokenizer_t* tok, xg_cache_pool_t** out);
void xg_cache_pool_destroy(xg_cache_pool_t* pool);
/* Size limit of the pool's device memory (Section 3.3: at the limit the least recently used entries
 * are evicted).  Entries are evicted in the batches they were built in, oldest use first, and only
 * once no live grammar uses any entry of the batch; a later compile rebuilds what it misses.
 * The limit counts the entries' bytes; the pool takes device memory in slabs (at most 64 MiB each)
 * and returns a slab when nothing in it is live.
 * max_bytes <= 0: no limit (the default).  May synchronise the device when it evicts. */
xg_status_t xg_cache_pool_set_limit(xg_cache_pool_t* pool, int64_t max_bytes);
/* Take `bytes` of device memory for the pool now (Section 3.5: what can be prepared before requests arrive
 * is).  Taking memory from the driver costs tens of microseconds per MiB; a pool that grows while grammars
 * compile pays that inside their compile times, a server that knows its cache budget pays it once at start-up.
 * The reservation is kept until the pool is destroyed and is used before any further memory is taken.
 * XG_ERR_OOM if the device has no room.  Synchronous. */
xg_status_t xg_cache_pool_reserve(xg_cache_pool_t* pool, int64_t bytes);
typedef struct {
  int64_t bytes;             /* bytes of cache entries held now (what the limit bounds) */
  int64_t reserved_bytes;    /* device memory the pool's slabs hold, grammars' own tables included */
  int64_t evicted_bytes;     /* total evicted so far */
  int64_t evicted_chunks;
  int32_t live_rules;        /* rule automata whose entries are in the pool */
  int32_t chunks;            /* batches of entries held now */
} xg_cache_pool_stats_t;
xg_status_t xg_cache_pool_stats(xg_cache_pool_t* pool, xg_cache_pool_stats_t* out);

typedef struct {
  uint32_t struct_size;       /* sizeof(xg_compile_options_t), for versioning */
  int32_t inline_max_states;  /* inline non-recursive rules whose automaton has at most this many
                                 states into their users; 0 = never; negative = default (16). */
  int32_t max_rule_states;    /* XG_ERR_CAPACITY if one rule's automaton grows past this.  <= 0 = default (1<<20). */
  int32_t build_cache;        /* 0 = front end only (tables, no device work).  Otherwise build. */
  int32_t no_state_compression; /* non-zero: build one cache entry per scannable state even where repetition
                                 state compression (Section 3.6) would let states share one. */
  int32_t jit;                /* non-zero: just-in-time cache (Section 3.5).  The compile builds only the
                                 jit_precompute costliest entries that the pool does not already hold; the others
                                 are built when a matcher first visits their state (xg_jit_service). */
  int32_t jit_precompute;     /* K of Section 3.5's configurable JIT: entries to build at compile time, the
                                 costliest first (cost = tokens that survive the state's first-byte test). */
  int64_t jit_arena_bytes;    /* size of the pool's first just-in-time arena (entries built inside the decode loop take
                                 their space from it on the device); when one fills up the next is twice as large.
                                 <= 0 = default (32 MiB).  Only the pool's first just-in-time compile sets it. */
  int32_t count_node_visits;  /* non-zero: the classification also counts the token bytes its walks consume
                                 (xg_grammar_stats_t.node_visits); statistics only, costs an atomic per warp. */
  int32_t repeat_threshold;   /* counted repetitions (Section 3.6): a bounded repetition X{l,r} with r >= this many iterations
                                 is kept as one copy of X whose Earley items carry the count k of finished iterations (the
                                 paper's parser state (R{l,r}, k)), so states and front-end time do not grow with r.
                                 0 = default (64); negative = never (every repetition is expanded into explicit states). */
  int32_t repeat_depth;       /* the longest token in bytes, for front-end-only compiles (tok == NULL); ignored when a
                                 tokenizer is given (its own longest token is used).  Without either, nothing is counted. */
  int32_t reserved;
} xg_compile_options_t;

/* ---- grammar compilation (Section 3.5 "compilation stage"; Sections 3.2, 3.3, 3.4) ---------
 * Parses `text` (EBNF with the TagDispatch intrinsic, a JSON schema, or a TagDispatch spec in
 * JSON), lowers it to one byte-level automaton per rule with byte-class and rule-reference edges
 * (Section 3.3), and fills the adaptive token mask cache on the GPU: for every scannable state
 * and every token, accepted / rejected / uncertain, stored as the smallest of accepted list,
 * rejected list or bitset, plus the uncertain list (Section 3.4).
 * tok == NULL (or opt->build_cache == 0): front end only; the result can be inspected with
 * xg_grammar_get_tables but cannot make matchers, and no CUDA call is made.
 * pool may be NULL (a private pool is used).  root_rule: EBNF only, NULL = "root".
 * Synchronous: the cache is complete when the call returns.
 * May be called from several host threads at once, also with one pool: the front ends run side
 * by side, the cache builds of one pool take turns (each thread must have the device current).
 * Errors: XG_ERR_PARSE, XG_ERR_UNSUPPORTED, XG_ERR_CAPACITY, XG_ERR_CUDA, XG_ERR_OOM. */
xg_status_t xg_compile_grammar(const xg_tokenizer_t* tok, xg_cache_pool_t* pool, xg_grammar_kind_t kind,
                               const char* text, size_t len, const char* root_rule,
                               const xg_compile_options_t* opt, void* stream, xg_grammar_t** out);
void xg_grammar_destroy(xg_grammar_t* g);

/* Flattened rule and byte-class tables (host copies, valid until the grammar is destroyed).
 * Rule r is an automaton over states; state s belongs to rule state_rule[s]; rule_start[r] is
 * its start state; state_final[s] != 0 marks accepting states.  Byte-class edges of s are
 * cedge_class/cedge_target[cedge_begin[s] .. cedge_begin[s+1]); rule-reference edges are
 * redge_rule/redge_target[redge_begin[s] .. redge_begin[s+1]).  Class c contains byte b iff bit
 * (b & 31) of class_bits[8*c + (b >> 5)] is set.  No rule accepts the empty string (references
 * to such rules have been bypassed); root_nullable says whether the root rule originally did.
 * A state is scannable iff it has at least one byte-class edge. */
typedef struct {
  int32_t n_rules, n_states, n_classes, n_class_edges, n_ref_edges;
  int32_t root_rule, root_nullable;
  const int32_t* rule_start;
  const int32_t* state_rule;
  const uint8_t* state_final;
  const int32_t* cedge_begin;
  const int32_t* cedge_class;
  const int32_t* cedge_target;
  const int32_t* redge_begin;
  const int32_t* redge_rule;
  const int32_t* redge_target;
  const uint32_t* class_bits;
  /* Counted repetitions (Section 3.6), NULL when the grammar has none.  rule_rep_lo/hi[r] != 0: rule r is X{lo,hi}
   * (1 <= lo <= hi) on the automaton of X, whose accepting states also carry copies of the start state's edges with
   * cedge_iter / redge_iter set ("the next iteration starts here").  An item of such a rule is (state, origin, k),
   * k = iterations finished before the current one: an iteration edge needs k + 1 < hi and leads to k + 1, the other
   * edges keep k, and the item is complete iff its state is accepting and k + 1 >= lo. */
  const int32_t* rule_rep_lo;
  const int32_t* rule_rep_hi;
  const uint8_t* cedge_iter;
  const uint8_t* redge_iter;
  int32_t n_records;          /* what the cache is indexed by: n_states, plus one record per class of counts for the states
                                 of counted rules (xg_grammar_record_of) */
} xg_grammar_tables_t;
xg_status_t xg_grammar_get_tables(const xg_grammar_t* g, xg_grammar_tables_t* host_view);

/* The cache record of (state, count): `state` itself for ordinary states; for a state of a counted rule the record of
 * the class its count falls into -- counts that no token of this vocabulary can tell apart, i.e. equally far (up to the
 * longest token's length) from both bounds, share one record and one cache entry (Section 3.6).
 * xg_grammar_get_cache_entry takes records.  XG_ERR_INVALID_ARG if the count is not below the rule's upper bound. */
xg_status_t xg_grammar_record_of(const xg_grammar_t* g, int32_t state, int32_t count, int32_t* record);

/* Structural hash of every rule (Section 3.3: Algorithm 1 bottom-up over the reference graph,
 * cycles refined as in Algorithm 2), the keys of the cross-grammar cache.  out: host, [n_rules].
 * Equal structures hash equally whatever the rule names and numbering; the pool additionally
 * compares canonical serialisations, so a collision can never share an entry. */
xg_status_t xg_grammar_get_rule_hashes(const xg_grammar_t* g, uint64_t* out);

/* Repetition state compression (Section 3.6), for repetitions below xg_compile_options_t.repeat_threshold.  Such an
 * R{l,r} is kept as explicit automaton states (the count k of the paper's state (R{l,r}, k) is the state itself), but
 * cache entries are built once per class of states that no token can tell apart: states of one rule whose automata
 * agree when unrolled `depth` edges deep.  With depth = the longest token in bytes their accepted / rejected /
 * uncertain sets are identical, so inside a repetition only the copies within `depth` of the bounds get entries of
 * their own.  out (host, [n_states]): for each state the smallest state of its class.  depth < 0: the tokenizer's
 * longest token (grammars compiled without a tokenizer: XG_ERR_INVALID_ARG).  A grammar with counted repetitions
 * (rule_rep_hi != NULL in its tables) answers XG_ERR_UNSUPPORTED: its records are the classes (xg_grammar_record_of).
 * Host work only. */
xg_status_t xg_grammar_get_state_classes(const xg_grammar_t* g, int32_t depth, int32_t* out);

/* One cache entry, copied to the host (valid until the next call on this grammar or its
 * destruction).  list = accepted ids (XG_STORE_ACCEPT_LIST) or rejected ids
 * (XG_STORE_REJECT_LIST), ascending; bitset = accepted bits (XG_STORE_BITSET), ceil(V/32) words;
 * uncertain = ascending ids.  Returns XG_ERR_INVALID_ARG if `state` is not scannable, or if a
 * just-in-time grammar has not built (and confirmed, see xg_jit_service) its entry yet.
 * Synchronises the device. */
typedef struct {
  int32_t state, kind;
  int32_t n_accepted, n_rejected, n_uncertain;
  int32_t n_list;
  const int32_t* list;
  const uint32_t* bitset;
  const int32_t* uncertain;
} xg_cache_entry_view_t;
xg_status_t xg_grammar_get_cache_entry(const xg_grammar_t* g, int32_t state, xg_cache_entry_view_t* host_view);

typedef struct {
  int32_t n_rules, n_states, n_scannable, n_classes;
  int32_t n_entries_built;      /* scannable states classified on the GPU by this compile */
  int32_t n_entries_reused;     /* scannable states served by the pool (Section 3.3) */
  int64_t pairs_classified;     /* n_entries_built * vocab_size */
  int64_t total_accepted, total_rejected, total_uncertain;   /* over this grammar's entries */
  int32_t kind_count[3];        /* entries per xg_store_kind_t */
  int32_t pad;
  int64_t cache_bytes;          /* device bytes of this grammar's entries (shared ones included) */
  double frontend_ms, cache_build_ms;   /* host front end; GPU classification + packing */
  int64_t total_checked;        /* uncertain tokens left after this grammar's lookahead narrowed the lists (Section 3.3):
                                   what the per-step check actually streams; <= total_uncertain */
  int64_t n_entries_shared;     /* scannable states that use the entry of an equivalent state of their rule
                                   (repetition state compression, Section 3.6) instead of one of their own */
  double classify_ms;           /* device time of the classification kernel alone (inside cache_build_ms) */
  int64_t node_visits;          /* with opt->count_node_visits: token bytes consumed by the classification walks of this
                                   compile, i.e. viable trie nodes visited without sharing between tokens (else 0) */
} xg_grammar_stats_t;
xg_status_t xg_grammar_stats(const xg_grammar_t* g, xg_grammar_stats_t* out);

/* ---- just-in-time cache build (Section 3.5) ------------------------------------------------
 * A grammar compiled with opt->jit starts with (nearly) no cache entries.  Masks are exact from the
 * first step on: while a scannable state of a matcher's current Earley set has no entry yet, the
 * fill kernel takes that request's mask from the plain definition (every token walked against the
 * full Earley state) and reports the state in a device-side ring.  xg_jit_service, called between
 * decode steps, reads the ring and gets the missing entries: from the pool if another grammar has
 * built them since (a cache hit), else by enqueueing the cache-build kernels on `stream`; the new
 * entries become visible to later fills in stream order.  States that are never visited are never
 * built.
 *   - The call never waits for the GPU unless wait != 0: it polls events, copies a few KB and
 *     enqueues kernels.  A miss reported by the fill of step t is picked up by the service call
 *     after step t+1 at the earliest, so a new state costs a few fallback steps.
 *   - wait != 0: also synchronises `stream` repeatedly until nothing is reported and nothing is in
 *     flight (what a caller does while the model prefills, and what tests use).
 *   - Use one stream for the fills, accepts and service calls of all just-in-time grammars of a
 *     pool, or order them with events: publishing an entry races with a fill running elsewhere.
 *   - Entries that arrive just in time get the grammar's lookahead narrowing like those of a full compile.
 * grammars: host array of n handles; those compiled without jit are skipped.  out may be NULL. */
typedef struct {
  int32_t n_built;        /* entries built just in time so far, over the given grammars (one per class of states) */
  int32_t n_pool_hits;    /* visited entries found in the pool instead of being built */
  int32_t n_in_flight;    /* entries whose build is enqueued and not yet confirmed */
  int32_t n_missing;      /* entries (classes of scannable states) still not built */
} xg_jit_stats_t;
xg_status_t xg_jit_service(xg_grammar_t* const* grammars, int32_t n, void* stream, int32_t wait, xg_jit_stats_t* out);

/* ---- matcher: one request's Earley state (Section 3.4) ------------------------------------ */
typedef struct {
  uint32_t struct_size;
  int32_t max_sets;    /* history capacity in Earley sets (one per accepted byte).  <= 0 = default (16384). */
  int32_t max_items;   /* history capacity in items.  <= 0 = default (4 * max_sets). */
} xg_matcher_options_t;
xg_status_t xg_matcher_create(const xg_grammar_t* g, const xg_matcher_options_t* opt, void* stream, xg_matcher_t** out);
xg_status_t xg_matcher_reset(xg_matcher_t* m, void* stream);
void xg_matcher_destroy(xg_matcher_t* m);
/* *out = 1 iff EOS has been accepted.  Synchronises `stream`. */
xg_status_t xg_matcher_is_terminated(const xg_matcher_t* m, void* stream, int32_t* out);

/* What the next xg_fill_next_token_bitmask has to stream for this matcher (for measurements): the
 * bytes of the cache entries it merges (bitsets in full, lists in full -- a block reads only its
 * slice of a list, but all blocks together read all of it), the uncertain candidates it tests
 * (12 bytes each: token rank, exit mask, and what is left at the first exit) and the row it writes.  List lengths and check
 * counts are the compile-time ones (entries that arrived just in time count with their whole
 * uncertain list).  Synchronises `stream`. */
typedef struct {
  int32_t n_merge, n_check, n_missing, pad;
  int64_t merge_bytes, check_tokens, check_bytes, row_bytes;
} xg_fill_work_t;
xg_status_t xg_matcher_next_fill_work(const xg_matcher_t* m, void* stream, xg_fill_work_t* out);

/* ---- per decode step ----------------------------------------------------------------------
 * xg_fill_next_token_bitmask: for each of `batch` matchers (host array of handles, all on one
 * tokenizer, grammars may differ) write its next-token bitmask into
 * bitmask_dev[i*row_stride_words .. +ceil(V/32)) (device).  Merge rule of the appendix on
 * XGrammar's cache: a token accepted by the cache of at least one current scannable state is
 * allowed; otherwise, if some cache calls it uncertain, it is checked against the matcher's full
 * Earley state; otherwise it is rejected.  EOS is allowed iff the root rule is complete.
 * (Just-in-time grammars: a request with an entry still missing gets the same mask from a walk of
 * the whole vocabulary against its full Earley state.)
 * Token walks run in small fixed arrays; a walk that does not fit them (an Earley set of more than 48
 * items, a token longer than 32 bytes) is redone exactly in a large per-matcher scratch, and a state
 * with more scannable entries than the step plan lists takes its mask from the plain definition, so
 * such states cost time, never a wrong or missing bit.  XG_ERR_CAPACITY is left for walks beyond that
 * scratch (2048 items, or more than 1024 such tokens in one step).
 * status_dev (device, [batch], may be NULL) receives XG_OK, XG_ERR_TERMINATED or XG_ERR_CAPACITY
 * per matcher; rows of matchers whose status is not XG_OK are all zero.
 * The first call with a list of matchers uploads the list (one asynchronous copy on `stream`); the
 * library caches the 64 most recently used lists, so a decode loop whose batch changes by a request
 * per step neither allocates nor synchronises the device once its largest batch has been seen.  Calls
 * on one tokenizer must be ordered among themselves (one stream, or events). */
xg_status_t xg_fill_next_token_bitmask(xg_matcher_t* const* matchers, int32_t batch,
                                       int32_t* bitmask_dev, int64_t row_stride_words,
                                       int32_t* status_dev, void* stream);

/* xg_fill_next_token_bitmask_static: the same result as xg_fill_next_token_bitmask, for callers
 * that must not allocate device memory inside their decode loop.  (The paper has no counterpart;
 * this is a deployment variant of the call above.)  A serving engine that has already handed all
 * free device memory to its own allocator, or that must keep its step free of the device-wide
 * synchronisation cudaMalloc / cudaFree imply, cannot use the call above for a batch it has not
 * seen before, because that call creates the batch's device-side request table and status words
 * on first use.  This variant keeps them in one fixed array that is part of the library image:
 * XG_STATIC_FILL_MAX_BATCH requests, 16 KiB, resident on every GPU that loads the library until
 * the process exits.  It never calls cudaMalloc, cudaFree or any allocating routine; the caller
 * still passes the bitmask (and optional status) buffers.
 *   - batch > XG_STATIC_FILL_MAX_BATCH returns XG_ERR_CAPACITY and does nothing.
 *   - The first call on each device looks up the array's device address; make that first call
 *     before any stream capture begins.
 *   - Every call on a device uses the same array: a small kernel at the head of each call rewrites
 *     the request table (which travels as a launch parameter, not through a host buffer) and clears
 *     the per-request words, so nothing is carried over from the previous call, but two calls whose
 *     GPU work overlaps (different streams) race; keep them on one stream or order them with events.
 * Arguments, layout, statuses and errors are otherwise those of xg_fill_next_token_bitmask. */
#define XG_STATIC_FILL_MAX_BATCH 1024
xg_status_t xg_fill_next_token_bitmask_static(xg_matcher_t* const* matchers, int32_t batch,
                                              int32_t* bitmask_dev, int64_t row_stride_words,
                                              int32_t* status_dev, void* stream);

/* xg_apply_token_bitmask: logits[r][v] = -inf where bit v of mask row r is 0 (Section 2.1), in
 * place, one pass.  logits_dev: device, [rows][logits_row_stride_elems] of dtype; every row must
 * start on a 16-byte boundary (XG_ERR_INVALID_ARG otherwise).  row_indices_dev (device, may be
 * NULL): the n_rows rows to touch (logits row = mask row = row_indices[i]); NULL = rows
 * 0..batch-1.  Elements whose bit is 1 are not modified in any way (NaN payloads and -0
 * survive); masked elements become the -inf bit pattern (0xFF800000 / 0xFF80) whatever they held. */
xg_status_t xg_apply_token_bitmask(void* logits_dev, xg_dtype_t dtype, int32_t batch, int32_t vocab_size,
                                   int64_t logits_row_stride_elems, const int32_t* bitmask_dev,
                                   int64_t mask_row_stride_words, const int32_t* row_indices_dev,
                                   int32_t n_rows, void* stream);

/* xg_accept_token: advance each matcher by its sampled token (Section 2.2 "trace the output";
 * scan / complete / predict of the appendix on Earley's algorithm).  token_ids_dev: device,
 * [batch].  status_dev (device, [batch], may be NULL): XG_OK; XG_ERR_TOKEN_REJECTED (state
 * unchanged); XG_ERR_TERMINATED; XG_ERR_CAPACITY (state unchanged).  Accepting EOS when the
 * root is complete terminates the matcher. */
xg_status_t xg_accept_token(xg_matcher_t* const* matchers, int32_t batch, const int32_t* token_ids_dev,
                            int32_t* status_dev, void* stream);

/* xg_accept_token_ex: xg_accept_token with one option.  restart_on_eos != 0: a request that
 * accepts the end-of-sequence token is put back into its initial state in the same launch (what
 * xg_matcher_reset would do in a launch of its own) instead of terminating -- for slots that
 * begin the next document of the same grammar at once.  restart_on_eos == 0 is xg_accept_token. */
xg_status_t xg_accept_token_ex(xg_matcher_t* const* matchers, int32_t batch, const int32_t* token_ids_dev,
                               int32_t* status_dev, int32_t restart_on_eos, void* stream);

/* xg_accept_token_and_fill_next_bitmask: xg_accept_token followed by xg_fill_next_token_bitmask
 * on the same batch, in one launch (Section 2.2: after a token is sampled the engine traces it
 * and generates the next step's mask; the two steps always follow each other in a decode loop).
 * The result is the one the two calls give in that order: accept_status_dev (device, [batch],
 * may be NULL) receives what xg_accept_token would report; a request whose token was rejected
 * keeps its state, and its mask row is the mask of that unchanged state; a request that
 * terminated gets an all-zero row and XG_ERR_TERMINATED in fill_status_dev (device, [batch], may
 * be NULL).  restart_on_eos != 0: a request that accepts the end-of-sequence token is put back
 * into its initial state (as by xg_matcher_reset) instead of terminating, and its row is the
 * mask of the grammar's start -- for slots that begin the next document of the same grammar at
 * once.  Where the vocabulary is too large for the one-launch fill the call enqueues the two
 * steps one after the other.  Other arguments, layout and errors: as in the two calls it
 * replaces. */
xg_status_t xg_accept_token_and_fill_next_bitmask(xg_matcher_t* const* matchers, int32_t batch,
                                                  const int32_t* token_ids_dev, int32_t* accept_status_dev,
                                                  int32_t restart_on_eos, int32_t* bitmask_dev,
                                                  int64_t row_stride_words, int32_t* fill_status_dev,
                                                  void* stream);

/* xg_fill_and_apply_token_bitmask: xg_fill_next_token_bitmask followed by xg_apply_token_bitmask on
 * rows 0..batch-1 of logits_dev, in one launch (Section 2.1: the mask is generated, then the logits of
 * the tokens it rules out are set to -inf).  Each request's mask row is applied to its logits row
 * straight from the on-chip copy the fill has just produced, so the mask is not read back from
 * memory, there is no kernel boundary between the two steps, and the rows of requests whose fill is
 * short are masked while other requests still check their uncertain tokens.  The results are exactly
 * those of the two calls in that order: bitmask_dev and status_dev as xg_fill_next_token_bitmask
 * writes them (the row of a request whose status is not XG_OK is all zero, so all of its logits
 * become -inf); logits as xg_apply_token_bitmask leaves them (same layout, alignment rule, dtype and
 * bit patterns; logits row i belongs to matchers[i]).  Where the vocabulary is too large for the
 * one-launch fill the call enqueues the steps one after the other. */
xg_status_t xg_fill_and_apply_token_bitmask(xg_matcher_t* const* matchers, int32_t batch,
                                            int32_t* bitmask_dev, int64_t row_stride_words,
                                            int32_t* status_dev, void* logits_dev, xg_dtype_t dtype,
                                            int64_t logits_row_stride_elems, void* stream);

#ifdef __cplusplus
}
#endif
#endif  /* XG_H_ */
