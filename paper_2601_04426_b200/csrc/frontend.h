// Host front end: grammar text -> one byte-level automaton per rule -> flat tables.
//
// The paper represents a grammar as several finite-state machines whose edges are character
// ranges, references to other machines, or epsilon (Section 3.3), and runs an Earley parser whose
// items are (machine state, start position) (Section 3.4).  This front end produces exactly that,
// normalised so the device loops stay table-driven:
//   * every rule is a deterministic automaton over bytes and rule references (no epsilon edges);
//   * no rule accepts the empty string (references to such rules are bypassed), so a rule
//     predicted at input position i can only complete at a later position;
//   * every state can reach an accepting state and every rule derives some string, so a
//     non-empty Earley set always means "viable prefix";
//   * small non-recursive rules are inlined into their users, which keeps more tokens decidable
//     inside one rule (fewer context-dependent tokens in the mask cache);
//   * TagDispatch (Section 3.2) becomes an ordinary rule whose automaton is the Aho-Corasick
//     automaton of the tags and stop strings, with a rule-reference edge per tag.
#pragma once

#include <cstdint>
#include <string>
#include <vector>

namespace xg {

struct FrontendError {
  int status;
  std::string message;
};

struct FrontendOptions {
  int inline_max_states = 16;
  int max_rule_states = 1 << 20;
  // Counted repetitions (Section 3.6).  A bounded repetition X{l,r} with r >= repeat_threshold becomes a rule of its
  // own whose automaton is X's with a loop back, and whose Earley items carry the count k of finished iterations;
  // the number of states no longer depends on r.  0 = never (every repetition is expanded into explicit states).
  // repeat_depth: the longest token in bytes; the count is only told apart where it is within repeat_depth + 1
  // iterations of a bound (see FlatGrammar::rep_depth).  Required (> 0) when repeat_threshold > 0.
  int repeat_threshold = 0;
  int repeat_depth = 0;
};

// bit 31 of a packed target: the new item's origin is the current set (the edge belongs to a rule
// predicted here) rather than the origin of the item that owns the list
constexpr uint32_t kSelfBit = 0x80000000u;
// Packed targets of edges that stay inside a counted-repetition rule (device view only): the new item keeps the
// count of the item that owns the edge (kRelBit), one more when the edge starts the next iteration (kIterBit).
constexpr uint32_t kRelBit = 0x40000000u, kIterBit = 0x20000000u;
constexpr uint32_t kTargetMask = 0x1FFFFFFFu;

struct FlatGrammar {
  int32_t n_rules = 0, n_states = 0, n_classes = 0;
  int32_t root_rule = 0, root_nullable = 0;
  int32_t max_expanded_repeat = 0;                 // the largest bound of a repetition that was expanded into explicit states
  std::vector<std::string> rule_names;
  std::vector<int32_t> rule_start, rule_kind;      // kind 1 = holds a TagDispatch automaton
  std::vector<int32_t> state_rule;
  std::vector<uint8_t> state_final;
  std::vector<int32_t> cedge_begin, cedge_class, cedge_target;
  std::vector<int32_t> redge_begin, redge_rule, redge_target;
  std::vector<uint32_t> class_bits;                // [n_classes][8]

  // Derived, for the device.  "Kernel" items are the ones created by scan or complete; items
  // created by predict are implied by these per-state lists:
  //   scan list of s  = own byte-class edges, then the byte-class edges of the start state of
  //                     every rule predicted (transitively) from s, flagged kSelfBit;
  //   wait list of s  = own rule-reference edges, then those of the predicted start states
  //                     (kSelfBit): who advances when rule r completes back into this set;
  //   gather list of s = the scannable states among s and its predicted start states (the
  //                     latter flagged kSelfBit, even when equal to s): the cache entries a
  //                     kernel item contributes to a step's mask.
  std::vector<int32_t> scan_begin, scan_own_end;
  std::vector<uint32_t> scan_class, scan_target;
  std::vector<int32_t> wait_begin;
  std::vector<uint32_t> wait_rule, wait_target;
  std::vector<int32_t> gather_begin, gather_state;
  // state_first[s] = bytes the scan list of s (own and predicted edges) can take; rule_follow[r] = bytes that can
  // come right after rule r completes, anywhere in this grammar (the lookahead of Section 3.3): the first bytes
  // of every state a reference to r leads to, plus, where that state is accepting, the follow set of its own rule
  std::vector<uint32_t> state_first, rule_follow;          // [S][8], [R][8]

  // Counted repetitions (Section 3.6: the parser state (R{l,r}, k)).  rule_rep_lo/hi[r] != 0 marks rule r as X{lo,hi}
  // (1 <= lo <= hi): its automaton is X's, and every accepting state of X also carries copies of the start state's
  // edges, flagged in cedge_iter / redge_iter ("the next iteration starts here").  An item of such a rule is
  // (state, origin, k), k = iterations finished before the current one: an iteration edge needs k + 1 < hi and
  // leads to k + 1, every other edge keeps k, and the item is complete iff its state is accepting and k + 1 >= lo.
  // Empty vectors: the grammar has no such rule.
  std::vector<int32_t> rule_rep_lo, rule_rep_hi;           // [R]
  std::vector<uint8_t> cedge_iter, redge_iter;             // parallel to cedge_class / redge_rule

  // Device view of a grammar with counted repetitions (`records`, built by expand_counted_rules): a state of a
  // counted rule appears once per class of counts that no token of at most rep_depth - 1 bytes can tell apart --
  // (min(max(lo - k - 1, 0), D), min(hi - k - 1, D)) with D = rep_depth -- as record
  // rep_rec_base[q - rep_first] + dl * (D + 1) + dr; acceptance and the iteration edges are then static per
  // record, and so is its cache entry.  In that view cedge_target / redge_target name the record of the class's
  // largest count (an ordinary automaton, which is what rule hashing and the pool see), cedge_word / redge_word
  // hold what the device follows: base state | kRelBit | kIterBit.  An item's state word is base state | k << rep_shift.
  int32_t rep_first = 0x7FFFFFFF, rep_shift = 31, rep_depth = 0, n_base_states = 0;
  std::vector<int32_t> rep_rec_base, rep_lo, rep_hi;       // per base state of a counted rule (q - rep_first)
  std::vector<uint32_t> cedge_word, redge_word;            // parallel to cedge_target / redge_target (records view only)
  std::vector<uint32_t> rec_word;                          // [S] records view: a state word that belongs to the record
};

enum GrammarKind { kEbnf = 0, kJsonSchema = 1, kTagDispatchJson = 2 };

// Throws FrontendError.
FlatGrammar compile_frontend(int kind, const std::string& text, const std::string& root, const FrontendOptions& opt);

// The device view of a grammar with counted repetitions (see FlatGrammar::rep_first); `g` itself when it has none.
FlatGrammar expand_counted_rules(const FlatGrammar& g);
// record of (base state q, count k) in the device view `records` of a grammar (q itself for ordinary states)
int32_t record_of(const FlatGrammar& records, int32_t q, int32_t k);

// Repetition state compression (Section 3.6): states of one rule that agree when their automata
// are unrolled `depth` edges deep share one cache entry.  Returns the class representative (the
// smallest such state) of every state.
std::vector<int32_t> bounded_equivalence(const FlatGrammar& g, int depth);

// The two text-to-text lowerings (exposed for tests and diagnostics).
std::string json_schema_to_ebnf(const std::string& schema_json, const std::string& root_name, const std::string& prefix);
std::string tag_dispatch_to_ebnf(const std::string& spec_json);

}  // namespace xg
