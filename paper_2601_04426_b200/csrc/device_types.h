// Plain structs shared by host code and kernels (all pointers are device pointers).
#pragma once
#include <cstddef>
#include <cstdint>

#include <vector_types.h>

namespace xg {

// Bounds-checking build (-DXG_DEBUG_BOUNDS): every index into a grammar table, the vocabulary arena, a request's
// chart or another block's shared memory is range-checked before use.  A check that fails records the first
// violation in a device word (what, index, limit) and makes the code skip the access -- it never traps.  The
// host reads the word with xg_debug_bounds_check.  Without the flag the checks compile to nothing.
enum : int {
  kBoundState = 1, kBoundScanEdge, kBoundWaitEdge, kBoundGather, kBoundClass, kBoundTokenRank, kBoundTokenBytes,
  kBoundChartSet, kBoundChartItem, kBoundWalkItem, kBoundPlanEntry, kBoundRowWord, kBoundClusterBlock, kBoundCheckList, kBoundEntry
};
#ifdef XG_DEBUG_BOUNDS
#define XG_BOUND(index, limit, what) ::xg::bound_ok((long long)(index), (long long)(limit), (what))
#else
#define XG_BOUND(index, limit, what) true
#endif

// Vocabulary, sorted by token bytes (trie order): tokens that share a prefix are adjacent, so
// neighbouring lanes of a warp walk the same automaton path for the shared prefix.
struct VocabDev {
  int32_t vocab_size;        // V
  int32_t n_words;           // ceil(V / 32)
  int32_t eos_id;            // -1 if none
  int32_t max_len;           // longest token in bytes
  const uint8_t* bytes;      // arena in rank order
  const uint32_t* offset;    // [V+1] by rank
  const int32_t* rank_to_id; // [V]
  const int32_t* id_to_rank; // [V]
  const uint8_t* never;      // [V] by rank: 1 = EOS, special or zero-length (never classified)
  uint32_t n_bytes;            // size of the arena (for the bounds-checking build)
  uint32_t pad;
  const uint32_t* first_rank;  // [257]: the tokens whose first byte is b are the ranks [first_rank[b], first_rank[b + 1])
                               // (zero-length tokens sort in front of first_rank[0])
};

// One adaptive cache entry (Section 3.4): the accepted/rejected split in its smallest form plus
// the uncertain tokens, the latter twice: by ascending id (set algebra) and by ascending rank
// (the order they are walked in).
struct EntryDev {
  const uint32_t* data;      // accepted ids | rejected ids | accepted bitset (n_words words)
  const uint32_t* unc_id;    // [n_unc] ascending token ids
  const uint32_t* unc_rank;  // [n_unc] ascending ranks
  const uint32_t* unc_exit;  // [n_unc] parallel to unc_rank: bit j = the token leaves the entry's rule after j bytes
  const uint32_t* unc_info;  // [n_unc] parallel to unc_rank: what the token has left at its first exit -- its byte there (what the
                             // context must scan) | the next byte << 8 | the number of bytes left (at most 255) << 16
  // The list the run-time check walks.  In the pool it is the uncertain list itself; a grammar
  // narrows it with its own lookahead (Section 3.3): exits whose next byte can never follow the
  // rule anywhere in that grammar are dropped, and tokens left without an exit with them.
  const uint32_t* chk_rank;
  const uint32_t* chk_exit;
  const uint32_t* chk_info;
  int32_t n_chk;
  int32_t pad2;
  int32_t kind;              // xg_store_kind_t; kEntryNotBuilt while a just-in-time grammar has not built it yet
  int32_t n_list;            // list length (0 for bitset)
  int32_t n_unc;
  int32_t n_acc;
};

constexpr int32_t kEntryNotBuilt = -1;

// Just-in-time cache build (Section 3.5): the fill kernels report the scannable states whose
// entry they found missing here; the host reads the ring between steps and builds them.
constexpr int kJitRingCap = 1024;
struct JitRing {                  // one per cache pool, shared by its just-in-time grammars
  uint32_t count;                 // reports so far (monotonic); report i is miss[i % kJitRingCap]
  uint32_t pad[3];
  int2 miss[kJitRingCap];         // (the grammar's slot in the pool, state)
};

// Everything a walk needs to know about one automaton state, in one 32-byte record (two 16-byte
// loads).  The scan list is scan_edge[scan_begin .. +n_scan) with the state's own edges first
// (n_own of them); its first edge is repeated inline, so the long literal chains of a schema
// grammar cost one load per byte.  A byte-class code is either a class id or, for a class of
// exactly one byte, kLiteral | byte (no bitset lookup).
struct __align__(16) StateRec {
  int32_t scan_begin;
  uint32_t n_own_n_scan;       // n_own | n_scan << 16
  int32_t wait_begin;
  uint32_t n_wait_n_gather;    // n_wait | n_gather << 16
  int32_t gather_begin;
  uint32_t info;               // rule id | accepting << 31
  uint32_t edge0_class, edge0_target;
};
constexpr uint32_t kLiteral = 0x80000000u;

struct GrammarDev {
  int32_t n_states, n_rules, n_classes;
  int32_t root_rule, root_nullable, root_start;
  const StateRec* state;          // [S]
  const uint2* scan_edge;         // (byte class, target); target bit 31: origin = the set being scanned
  const uint2* wait_edge;         // (awaited rule, target); target bit 31: origin = the set the rule started in
  const int32_t* gather_state;    // bit 31: a predicted start state (its items begin in the current set)
  const uint32_t* class_bits;     // [C][8]
  const uint32_t* state_first;    // [S][8] bytes that the state's scan list (own and predicted edges) can take
  const uint32_t* rule_follow;    // [R][8] bytes that can follow a completed rule somewhere in this grammar
  const EntryDev* entries;        // [S]; meaningful for scannable states
  JitRing* miss_ring;             // just-in-time grammars only (else nullptr)
  int32_t jit_slot;               // this grammar's number in the ring's reports
  int32_t n_scan_edges, n_wait_edges, n_gather;      // table sizes (for the bounds-checking build)
  // Counted repetitions (Section 3.6: the parser state (R{l,r}, k)).  An item's state word is state | k << rep_shift;
  // words below rep_first are ordinary states (k = 0) and index the tables directly.  A state q >= rep_first belongs
  // to a counted rule and has one record (tables, cache entry) per class of counts:
  //   rep_state[q - rep_first] = (first record, lo, hi, -),  record = first + dl * (rep_depth + 1) + dr,
  //   dl = min(max(lo - k - 1, 0), rep_depth), dr = min(hi - k - 1, rep_depth).
  // Edge targets inside such a rule carry kRel (keep the count) and kIter (one more).  rec_word[record] is a state
  // word of the record's class (the item a cache entry is classified from).  No counted rule: rep_first = INT32_MAX.
  int32_t rep_first, rep_shift, rep_depth, n_words_states;     // n_words_states: states before the records were written out
  const int4* rep_state;
  const uint32_t* rec_word;
};

// What the next mask needs from the current Earley set, worked out once when the set is made
// (by accept or reset) instead of by every block of the fill kernels:
//   * the cache entries to merge (scannable states of the set, predicted ones included);
//   * the entries that have uncertain tokens, as (state, origin) pairs, with for each the
//     continuation set -- what the chart looks like right after that state's rule completes --
//     and the bytes that set can scan;
//   * whether EOS is allowed.
constexpr int kPlanMergeMax = 64;
constexpr int kPlanCheckMax = 32;
constexpr int kContCap = 16;
constexpr int kPlanMissingMax = 8;
struct __align__(16) StepPlan {
  int32_t n_merge, n_check, eos_ok, overflow;
  uint32_t cont_first[kPlanCheckMax][8];     // read and written as 16-byte vectors: keep 16-byte aligned
  uint32_t cont_st[kPlanCheckMax][kContCap];
  int32_t cont_org[kPlanCheckMax][kContCap];
  int32_t merge_state[kPlanMergeMax];
  int32_t check_state[kPlanCheckMax];
  int32_t check_origin[kPlanCheckMax];
  int32_t cont_cnt[kPlanCheckMax];
  int32_t check_cum[kPlanCheckMax + 1];      // running totals of uncertain tokens
  // just-in-time grammars: scannable states of the current set whose entry is not built yet.  While there are any,
  // the step's mask comes from walking the whole vocabulary against the full Earley state (the plain definition).
  int32_t n_missing;                         // may exceed kPlanMissingMax; the first kPlanMissingMax are listed
  int32_t missing_state[kPlanMissingMax];
};
static_assert(offsetof(StepPlan, cont_first) % 16 == 0, "cont_first must be 16-byte aligned");

// One request's Earley chart.  Only "kernel" items (made by scan or complete) are stored; the
// predicted items of a set are implied by the grammar's per-state lists.
struct MatcherDev {
  const GrammarDev* grammar;
  uint32_t* item_state;
  int32_t* item_origin;
  int32_t* set_begin;        // [cap_sets + 1]
  int32_t n_sets, n_items;
  int32_t cap_sets, cap_items;
  int32_t terminated;
  int32_t slow_n;            // tokens queued for the exact slow walk by the fill that is running (reset by every fill)
  StepPlan* plan;
  // Exact slow path (one user at a time): a token walk that does not fit the fixed per-thread arrays -- more than
  // kFastCap items, or a token beyond kFastMaxBytes bytes -- is redone here, up to kSlowCap items and 255 bytes.
  uint32_t* slow_st;         // [kSlowCap]
  int32_t* slow_org;         // [kSlowCap]
  int32_t* slow_lsb;         // [257]
  int32_t* slow_q;           // [kSlowQueue] token ranks waiting for a slow walk
};
constexpr int kSlowQueue = 1024;

constexpr uint32_t kSelf = 0x80000000u;
constexpr uint32_t kRel = 0x40000000u, kIter = 0x20000000u, kTarget = 0x1FFFFFFFu;

}  // namespace xg
