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
};

// bit 31 of a packed target: the new item's origin is the current set (the edge belongs to a rule
// predicted here) rather than the origin of the item that owns the list
constexpr uint32_t kSelfBit = 0x80000000u;

struct FlatGrammar {
  int32_t n_rules = 0, n_states = 0, n_classes = 0;
  int32_t root_rule = 0, root_nullable = 0;
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
};

enum GrammarKind { kEbnf = 0, kJsonSchema = 1, kTagDispatchJson = 2 };

// Throws FrontendError.
FlatGrammar compile_frontend(int kind, const std::string& text, const std::string& root, const FrontendOptions& opt);

// Repetition state compression (Section 3.6): states of one rule that agree when their automata
// are unrolled `depth` edges deep share one cache entry.  Returns the class representative (the
// smallest such state) of every state.
std::vector<int32_t> bounded_equivalence(const FlatGrammar& g, int depth);

// The two text-to-text lowerings (exposed for tests and diagnostics).
std::string json_schema_to_ebnf(const std::string& schema_json, const std::string& root_name, const std::string& prefix);
std::string tag_dispatch_to_ebnf(const std::string& spec_json);

}  // namespace xg
