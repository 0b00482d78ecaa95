// CPU ORACLE -- TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, obviously-correct implementation of what the token-mask path computes.  It is
// used by the tests, by the smoke check and by the benchmark's CPU-baseline leg, and by nothing
// else: the library under csrc/ neither links nor calls it, and this file includes nothing from
// there.  It is not tuned for speed.
//
// What it computes, by definition rather than by the accelerated method:
//   * Earley recognition over bytes (paper Section 3.4 and the appendix "Earley's Parsing
//     Algorithm": an item is a rule, a position inside it and the input position where the rule
//     began; the operations are predict, scan, complete).  The paper's formal table is not
//     available, so this is the textbook recogniser, with the closure run to a fixpoint.
//   * The token mask (Section 2.1): token t is allowed iff feeding its bytes one at a time from
//     the current chart leaves a non-empty item set after every byte.  With every rule
//     productive, "non-empty set" is "viable prefix".  EOS is allowed iff the root rule is
//     complete with origin 0.  Special and zero-length tokens are never allowed.
//   * Mask application (Section 2.1): disallowed logits become -inf.
//   * TagDispatch (Section 3.2) as its plain definition: free text while tracking the longest
//     suffix that is a prefix of a tag/stop string (string comparison, no automaton); a completed
//     tag switches to its sub-grammar; when that completes, back to free text; a stop string
//     ends the construct; with no stop strings it may end at any byte while dispatching.
//   * On the flattened tables a grammar compiler exports (plain data), the accepted / rejected /
//     uncertain classification of a token at one scannable state (Section 3.4, appendix
//     "Adaptive Token Mask cache Generation Algorithm") and the run-time merge rule of that
//     appendix, both written out directly.
//
// Parity status: every function here is pinned by tests/test_oracle_*.py (brute-force string
// enumeration against an independent membership search, Python's `re` on regular grammars,
// `json.loads` on the any-JSON grammar, hand-worked masks, closed forms and invariants).
//
// Grammar text: rules `name ::= body`; body uses "literals" (UTF-8 text; escapes \n \t \r \\ \"
// \' \/ \xHH raw byte, \uHHHH, \UHHHHHHHH), [classes] of code points with ranges and ^ negation
// (escapes as above plus \] \- \^; \xHH is code point HH), rule names, ( ), |, postfix * + ?
// {m} {m,} {m,n}, `#` comments, and TagDispatch(("tag", rule), ..., stop_strs=("s", ...)).
// A class matches one well-formed UTF-8 encoded scalar value (no surrogates, no overlongs).

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <map>
#include <stdexcept>
#include <string>
#include <thread>
#include <vector>

namespace {

// ------------------------------------------------------------------------------------------
// grammar
// ------------------------------------------------------------------------------------------

struct CpRange { uint32_t lo, hi; };
enum SymKind { SYM_BYTE = 0, SYM_CPSET = 1, SYM_NT = 2, SYM_TD = 3 };
struct Sym { int kind; int arg; };
struct Alt { int rule; std::vector<Sym> syms; };

struct TagDispatch {
  std::vector<std::string> tags;
  std::vector<std::string> tag_rule_name;
  std::vector<int> tag_rule;
  std::vector<char> tag_dead;
  std::vector<std::string> stops;
  std::vector<std::string> prefixes;          // every proper prefix of every tag / stop string
  std::map<std::string, int> prefix_id;
};

struct Grammar {
  std::vector<std::string> names;
  std::map<std::string, int> name_id;
  std::vector<std::vector<int>> rule_alts;
  std::vector<Alt> alts;
  std::vector<std::vector<CpRange>> cpsets;
  std::vector<TagDispatch> tds;
  int root = -1;
};

struct Node {
  enum Type { STR, CLASS, REF, SEQ, ALT, STAR, PLUS, OPT, REP, TD } type = SEQ;
  std::string bytes;
  std::vector<CpRange> ranges;
  std::string name;
  std::vector<Node> kids;
  int lo = 0, hi = 0;     // REP bounds; hi < 0 = unbounded
  TagDispatch td;
};

void append_utf8(std::string& out, uint32_t cp) {
  if (cp < 0x80) out.push_back((char)cp);
  else if (cp < 0x800) { out.push_back((char)(0xC0 | (cp >> 6))); out.push_back((char)(0x80 | (cp & 0x3F))); }
  else if (cp < 0x10000) { out.push_back((char)(0xE0 | (cp >> 12))); out.push_back((char)(0x80 | ((cp >> 6) & 0x3F))); out.push_back((char)(0x80 | (cp & 0x3F))); }
  else { out.push_back((char)(0xF0 | (cp >> 18))); out.push_back((char)(0x80 | ((cp >> 12) & 0x3F))); out.push_back((char)(0x80 | ((cp >> 6) & 0x3F))); out.push_back((char)(0x80 | (cp & 0x3F))); }
}

class Parser {
 public:
  explicit Parser(const std::string& text) : s_(text) {}

  std::vector<std::pair<std::string, Node>> parse_grammar() {
    std::vector<std::pair<std::string, Node>> rules;
    skip();
    while (pos_ < s_.size()) {
      std::string name = ident();
      if (name.empty()) fail("expected a rule name");
      skip();
      if (s_.compare(pos_, 3, "::=") != 0) fail("expected ::= after rule name " + name);
      pos_ += 3;
      rules.emplace_back(name, alternation());
      skip();
    }
    return rules;
  }

 private:
  const std::string& s_;
  size_t pos_ = 0;

  [[noreturn]] void fail(const std::string& msg) {
    throw std::runtime_error("EBNF: " + msg + " at offset " + std::to_string(pos_));
  }
  void skip() {
    while (pos_ < s_.size()) {
      char c = s_[pos_];
      if (c == ' ' || c == '\t' || c == '\n' || c == '\r') ++pos_;
      else if (c == '#') { while (pos_ < s_.size() && s_[pos_] != '\n') ++pos_; }
      else break;
    }
  }
  static bool ident_start(char c) { return (c >= 'a' && c <= 'z') || (c >= 'A' && c <= 'Z') || c == '_'; }
  static bool ident_char(char c) { return ident_start(c) || (c >= '0' && c <= '9'); }
  std::string ident() {
    size_t p = pos_;
    if (p < s_.size() && ident_start(s_[p])) { ++p; while (p < s_.size() && ident_char(s_[p])) ++p; }
    std::string out = s_.substr(pos_, p - pos_);
    pos_ = p;
    return out;
  }
  // true when the upcoming identifier opens a new rule (`name ::=`)
  bool at_rule_head() {
    size_t save = pos_;
    std::string name = ident();
    bool head = false;
    if (!name.empty()) { skip(); head = s_.compare(pos_, 3, "::=") == 0; }
    pos_ = save;
    return head;
  }
  int hexval(char c) {
    if (c >= '0' && c <= '9') return c - '0';
    if (c >= 'a' && c <= 'f') return c - 'a' + 10;
    if (c >= 'A' && c <= 'F') return c - 'A' + 10;
    fail("bad hex digit");
  }
  uint32_t hex(int n) {
    uint32_t v = 0;
    for (int i = 0; i < n; ++i) { if (pos_ >= s_.size()) fail("truncated escape"); v = v * 16 + hexval(s_[pos_++]); }
    return v;
  }
  uint32_t source_cp() {     // decode one UTF-8 character of the grammar text
    unsigned char c = (unsigned char)s_[pos_++];
    if (c < 0x80) return c;
    int n = c >= 0xF0 ? 3 : c >= 0xE0 ? 2 : 1;
    uint32_t cp = c & (0x3F >> n);
    for (int i = 0; i < n; ++i) { if (pos_ >= s_.size()) fail("bad UTF-8 in grammar text"); cp = (cp << 6) | ((unsigned char)s_[pos_++] & 0x3F); }
    return cp;
  }
  // after a backslash: returns true and a code point, or (raw=true) a raw byte for \x in strings
  uint32_t escape(bool in_class, bool* raw) {
    *raw = false;
    if (pos_ >= s_.size()) fail("truncated escape");
    char c = s_[pos_++];
    switch (c) {
      case 'n': return '\n'; case 't': return '\t'; case 'r': return '\r';
      case '\\': return '\\'; case '"': return '"'; case '\'': return '\''; case '/': return '/';
      case 'x': *raw = !in_class; return hex(2);
      case 'u': return hex(4);
      case 'U': return hex(8);
      case ']': case '-': case '^': if (in_class) return (uint32_t)c; break;
      default: break;
    }
    fail(std::string("unknown escape \\") + c);
  }
  std::string string_literal() {
    ++pos_;   // opening quote
    std::string out;
    while (true) {
      if (pos_ >= s_.size()) fail("unterminated string");
      char c = s_[pos_];
      if (c == '"') { ++pos_; break; }
      if (c == '\\') { ++pos_; bool raw; uint32_t v = escape(false, &raw); if (raw) out.push_back((char)v); else append_utf8(out, v); }
      else { out.push_back(c); ++pos_; }
    }
    return out;
  }
  Node char_class() {
    ++pos_;   // '['
    Node n; n.type = Node::CLASS;
    bool neg = false;
    if (pos_ < s_.size() && s_[pos_] == '^') { neg = true; ++pos_; }
    std::vector<CpRange> rs;
    while (true) {
      if (pos_ >= s_.size()) fail("unterminated class");
      if (s_[pos_] == ']') { ++pos_; break; }
      uint32_t lo;
      bool raw;
      if (s_[pos_] == '\\') { ++pos_; lo = escape(true, &raw); } else lo = source_cp();
      uint32_t hi = lo;
      if (pos_ + 1 < s_.size() && s_[pos_] == '-' && s_[pos_ + 1] != ']') {
        ++pos_;
        if (s_[pos_] == '\\') { ++pos_; hi = escape(true, &raw); } else hi = source_cp();
        if (hi < lo) fail("reversed range in class");
      }
      rs.push_back({lo, hi});
    }
    // normalise: sort, merge, negate over [0, 0x10FFFF]
    std::sort(rs.begin(), rs.end(), [](const CpRange& a, const CpRange& b) { return a.lo < b.lo; });
    std::vector<CpRange> merged;
    for (auto r : rs) {
      if (!merged.empty() && r.lo <= merged.back().hi + 1) merged.back().hi = std::max(merged.back().hi, r.hi);
      else merged.push_back(r);
    }
    if (neg) {
      std::vector<CpRange> inv;
      uint32_t next = 0;
      for (auto r : merged) { if (r.lo > next) inv.push_back({next, r.lo - 1}); next = r.hi + 1; }
      if (next <= 0x10FFFF) inv.push_back({next, 0x10FFFF});
      merged = inv;
    }
    n.ranges = merged;
    return n;
  }
  int integer() {
    skip();
    size_t p = pos_;
    int v = 0;
    while (pos_ < s_.size() && s_[pos_] >= '0' && s_[pos_] <= '9') { v = v * 10 + (s_[pos_] - '0'); ++pos_; if (v > 1000000) fail("repetition bound too large"); }
    if (p == pos_) fail("expected an integer");
    return v;
  }
  void expect(char c) { skip(); if (pos_ >= s_.size() || s_[pos_] != c) fail(std::string("expected '") + c + "'"); ++pos_; }
  std::vector<std::string> string_tuple() {
    std::vector<std::string> out;
    expect('(');
    skip();
    while (pos_ < s_.size() && s_[pos_] != ')') {
      if (s_[pos_] != '"') fail("expected a string");
      out.push_back(string_literal());
      skip();
      if (pos_ < s_.size() && s_[pos_] == ',') { ++pos_; skip(); }
    }
    expect(')');
    return out;
  }
  Node tag_dispatch() {
    Node n; n.type = Node::TD;
    expect('(');
    skip();
    while (pos_ < s_.size() && s_[pos_] != ')') {
      if (s_[pos_] == '(') {
        ++pos_; skip();
        if (pos_ >= s_.size() || s_[pos_] != '"') fail("expected a tag string");
        std::string tag = string_literal();
        if (tag.empty()) fail("empty tag");
        expect(',');
        skip();
        std::string rule = ident();
        if (rule.empty()) fail("expected a rule name in TagDispatch");
        expect(')');
        n.td.tags.push_back(tag);
        n.td.tag_rule_name.push_back(rule);
      } else {
        std::string key = ident();
        if (key != "stop_strs") fail("unknown TagDispatch argument " + key);
        expect('=');
        n.td.stops = string_tuple();
        for (auto& st : n.td.stops) if (st.empty()) fail("empty stop string");
      }
      skip();
      if (pos_ < s_.size() && s_[pos_] == ',') { ++pos_; skip(); }
    }
    expect(')');
    return n;
  }
  Node alternation() {
    Node alt; alt.type = Node::ALT;
    while (true) {
      alt.kids.push_back(sequence());
      skip();
      if (pos_ < s_.size() && s_[pos_] == '|') { ++pos_; continue; }
      break;
    }
    return alt;
  }
  Node sequence() {
    Node seq; seq.type = Node::SEQ;
    while (true) {
      skip();
      if (pos_ >= s_.size()) break;
      char c = s_[pos_];
      if (c == '|' || c == ')') break;
      if (ident_start(c) && at_rule_head()) break;
      Node atom;
      if (c == '"') { atom.type = Node::STR; atom.bytes = string_literal(); }
      else if (c == '[') atom = char_class();
      else if (c == '(') { ++pos_; atom = alternation(); expect(')'); }
      else if (ident_start(c)) {
        std::string name = ident();
        if (name == "TagDispatch") atom = tag_dispatch();
        else { atom.type = Node::REF; atom.name = name; }
      } else fail(std::string("unexpected character '") + c + "'");
      // postfix operators
      while (true) {
        skip();
        if (pos_ >= s_.size()) break;
        char q = s_[pos_];
        Node wrap;
        if (q == '*') { wrap.type = Node::STAR; ++pos_; }
        else if (q == '+') { wrap.type = Node::PLUS; ++pos_; }
        else if (q == '?') { wrap.type = Node::OPT; ++pos_; }
        else if (q == '{') {
          ++pos_;
          wrap.type = Node::REP;
          wrap.lo = integer();
          wrap.hi = wrap.lo;
          skip();
          if (pos_ < s_.size() && s_[pos_] == ',') {
            ++pos_; skip();
            if (pos_ < s_.size() && s_[pos_] == '}') wrap.hi = -1; else wrap.hi = integer();
          }
          expect('}');
          if (wrap.hi >= 0 && wrap.hi < wrap.lo) fail("repetition upper bound below lower bound");
        } else break;
        wrap.kids.push_back(atom);
        atom = wrap;
      }
      seq.kids.push_back(atom);
    }
    return seq;
  }
};

class Lowering {
 public:
  explicit Lowering(Grammar& g) : g_(g) {}

  int new_rule(const std::string& name) {
    int id = (int)g_.names.size();
    g_.names.push_back(name);
    g_.rule_alts.emplace_back();
    return id;
  }
  void add_alt(int rule, const std::vector<Sym>& syms) {
    g_.rule_alts[rule].push_back((int)g_.alts.size());
    g_.alts.push_back({rule, syms});
  }
  void lower_rule(int rule, const Node& alternation) {
    for (const Node& seq : alternation.kids) {
      std::vector<Sym> syms;
      lower(seq, syms);
      add_alt(rule, syms);
    }
  }
  // append symbols deriving exactly L(n)
  void lower(const Node& n, std::vector<Sym>& out) {
    switch (n.type) {
      case Node::STR:
        for (unsigned char c : n.bytes) out.push_back({SYM_BYTE, (int)c});
        break;
      case Node::CLASS:
        g_.cpsets.push_back(n.ranges);
        out.push_back({SYM_CPSET, (int)g_.cpsets.size() - 1});
        break;
      case Node::REF: {
        auto it = g_.name_id.find(n.name);
        if (it == g_.name_id.end()) throw std::runtime_error("EBNF: undefined rule " + n.name);
        out.push_back({SYM_NT, it->second});
        break;
      }
      case Node::SEQ:
        for (const Node& k : n.kids) lower(k, out);
        break;
      case Node::ALT: {
        if (n.kids.size() == 1) { lower(n.kids[0], out); break; }
        int r = new_rule("$group" + std::to_string(g_.names.size()));
        lower_rule(r, n);
        out.push_back({SYM_NT, r});
        break;
      }
      case Node::STAR: {          // S ::= (empty) | S X
        int r = new_rule("$star" + std::to_string(g_.names.size()));
        add_alt(r, {});
        std::vector<Sym> syms{{SYM_NT, r}};
        lower(n.kids[0], syms);
        add_alt(r, syms);
        out.push_back({SYM_NT, r});
        break;
      }
      case Node::PLUS: {          // P ::= X | P X
        int r = new_rule("$plus" + std::to_string(g_.names.size()));
        std::vector<Sym> one;
        lower(n.kids[0], one);
        add_alt(r, one);
        std::vector<Sym> more{{SYM_NT, r}};
        lower(n.kids[0], more);
        add_alt(r, more);
        out.push_back({SYM_NT, r});
        break;
      }
      case Node::OPT: {           // O ::= (empty) | X
        int r = new_rule("$opt" + std::to_string(g_.names.size()));
        add_alt(r, {});
        std::vector<Sym> syms;
        lower(n.kids[0], syms);
        add_alt(r, syms);
        out.push_back({SYM_NT, r});
        break;
      }
      case Node::REP: {           // X{lo,hi}: lo copies, then hi-lo nested optional copies (or X*)
        for (int i = 0; i < n.lo; ++i) lower(n.kids[0], out);
        if (n.hi < 0) {
          Node star; star.type = Node::STAR; star.kids.push_back(n.kids[0]);
          lower(star, out);
        } else {
          int inner = -1;       // O_1 ::= (empty) | X ; O_k ::= (empty) | X O_{k-1}
          for (int k = 0; k < n.hi - n.lo; ++k) {
            int r = new_rule("$rep" + std::to_string(g_.names.size()));
            add_alt(r, {});
            std::vector<Sym> syms;
            lower(n.kids[0], syms);
            if (inner >= 0) syms.push_back({SYM_NT, inner});
            add_alt(r, syms);
            inner = r;
          }
          if (inner >= 0) out.push_back({SYM_NT, inner});
        }
        break;
      }
      case Node::TD: {
        TagDispatch td = n.td;
        for (auto& rn : td.tag_rule_name) {
          auto it = g_.name_id.find(rn);
          if (it == g_.name_id.end()) throw std::runtime_error("EBNF: undefined rule " + rn);
          td.tag_rule.push_back(it->second);
        }
        td.tag_dead.assign(td.tags.size(), 0);
        auto add_prefixes = [&](const std::string& p) {
          for (size_t l = 0; l < p.size(); ++l) {
            std::string pre = p.substr(0, l);
            if (!td.prefix_id.count(pre)) { td.prefix_id[pre] = (int)td.prefixes.size(); td.prefixes.push_back(pre); }
          }
        };
        add_prefixes("x");        // guarantees the empty prefix has id 0
        for (auto& t : td.tags) add_prefixes(t);
        for (auto& t : td.stops) add_prefixes(t);
        g_.tds.push_back(td);
        out.push_back({SYM_TD, (int)g_.tds.size() - 1});
        break;
      }
    }
  }

 private:
  Grammar& g_;
};

bool cpset_nonempty(const std::vector<CpRange>& set, uint32_t lo, uint32_t hi);

// drop alternatives that can never derive a byte string, so that "item set non-empty" means
// "the bytes read so far are a prefix of some sentence"
void prune_unproductive(Grammar& g) {
  std::vector<char> productive(g.names.size(), 0);
  auto sym_ok = [&](const Sym& s) {
    switch (s.kind) {
      case SYM_BYTE: return true;
      case SYM_CPSET: return cpset_nonempty(g.cpsets[s.arg], 0, 0x10FFFF);
      case SYM_NT: return productive[s.arg] != 0;
      default: return true;       // TagDispatch always derives something (free text)
    }
  };
  bool changed = true;
  while (changed) {
    changed = false;
    for (size_t r = 0; r < g.names.size(); ++r) {
      if (productive[r]) continue;
      for (int a : g.rule_alts[r]) {
        bool ok = true;
        for (const Sym& s : g.alts[a].syms) ok = ok && sym_ok(s);
        if (ok) { productive[r] = 1; changed = true; break; }
      }
    }
  }
  for (size_t r = 0; r < g.names.size(); ++r) {
    std::vector<int> keep;
    for (int a : g.rule_alts[r]) {
      bool ok = true;
      for (const Sym& s : g.alts[a].syms) ok = ok && sym_ok(s);
      if (ok) keep.push_back(a);
    }
    g.rule_alts[r] = keep;
  }
  for (auto& td : g.tds)
    for (size_t j = 0; j < td.tags.size(); ++j) td.tag_dead[j] = !productive[td.tag_rule[j]];
}

Grammar* grammar_from_ebnf(const std::string& text, const std::string& root) {
  Parser p(text);
  auto rules = p.parse_grammar();
  if (rules.empty()) throw std::runtime_error("EBNF: no rules");
  Grammar* g = new Grammar();
  try {
    Lowering low(*g);
    for (auto& r : rules) {
      if (g->name_id.count(r.first)) throw std::runtime_error("EBNF: rule defined twice: " + r.first);
      g->name_id[r.first] = low.new_rule(r.first);
    }
    for (auto& r : rules) low.lower_rule(g->name_id[r.first], r.second);
    auto it = g->name_id.find(root);
    if (it == g->name_id.end()) throw std::runtime_error("EBNF: root rule not found: " + root);
    g->root = it->second;
    prune_unproductive(*g);
  } catch (...) { delete g; throw; }
  return g;
}

// ------------------------------------------------------------------------------------------
// UTF-8: "does the class contain a scalar value whose encoding starts with these bytes?"
// ------------------------------------------------------------------------------------------

bool cpset_nonempty(const std::vector<CpRange>& set, uint32_t lo, uint32_t hi) {
  if (hi > 0x10FFFF) hi = 0x10FFFF;
  for (const CpRange& r : set) {
    uint32_t a = std::max(lo, r.lo), b = std::min(hi, r.hi);
    if (a > b) continue;
    if (a <= 0xD7FF) return true;                 // part below the surrogate block
    if (b >= 0xE000 && std::max(a, (uint32_t)0xE000) <= b) return true;
  }
  return false;
}

const uint32_t kLenLo[5] = {0, 0x0, 0x80, 0x800, 0x10000};
const uint32_t kLenHi[5] = {0, 0x7F, 0x7FF, 0xFFFF, 0x10FFFF};

// aux packs a partly read character: total length (bits 28..30), bytes seen (24..26), value bits
inline uint32_t pack_aux(int total, int seen, uint32_t acc) { return ((uint32_t)total << 28) | ((uint32_t)seen << 24) | acc; }

// returns 0 = byte refused, 1 = character still incomplete (new aux), 2 = character complete
int cpset_step(const std::vector<CpRange>& set, uint32_t aux, uint8_t b, uint32_t* new_aux) {
  int total, seen;
  uint32_t acc;
  if (aux == 0) {
    if (b < 0x80) return cpset_nonempty(set, b, b) ? 2 : 0;
    if (b >= 0xC0 && b <= 0xDF) { total = 2; acc = b & 0x1F; }
    else if (b >= 0xE0 && b <= 0xEF) { total = 3; acc = b & 0x0F; }
    else if (b >= 0xF0 && b <= 0xF7) { total = 4; acc = b & 0x07; }
    else return 0;
    seen = 1;
  } else {
    total = (aux >> 28) & 7; seen = (aux >> 24) & 7; acc = aux & 0xFFFFFF;
    if (b < 0x80 || b > 0xBF) return 0;
    acc = (acc << 6) | (b & 0x3F);
    ++seen;
  }
  int rem = total - seen;
  uint32_t lo = acc << (6 * rem), hi = lo | ((1u << (6 * rem)) - 1);
  lo = std::max(lo, kLenLo[total]);
  hi = std::min(hi, kLenHi[total]);
  if (lo > hi || !cpset_nonempty(set, lo, hi)) return 0;
  if (rem == 0) return 2;
  *new_aux = pack_aux(total, seen, acc);
  return 1;
}

// ------------------------------------------------------------------------------------------
// Earley recogniser
// ------------------------------------------------------------------------------------------

enum ItemKind { IT_NORMAL = 0, IT_TDFREE = 1, IT_TDWAIT = 2, IT_TDDONE = 3 };
// NORMAL: a = alternative, b = dot, aux = partly read character.
// TDFREE: a = TagDispatch id, b = id of the tracked suffix.  TDWAIT: b = tag index (sub-grammar
// running).  TDDONE: a stop string was just read.
struct Item { int kind, a, b, origin; uint32_t aux; };
inline bool same(const Item& x, const Item& y) { return x.kind == y.kind && x.a == y.a && x.b == y.b && x.origin == y.origin && x.aux == y.aux; }
typedef std::vector<Item> Set;

inline bool add_item(Set& s, const Item& it) {
  for (const Item& x : s) if (same(x, it)) return false;
  s.push_back(it);
  return true;
}

// a chart seen as an immutable base followed by private extra sets (used while probing a token)
struct View {
  const std::vector<Set>* base;
  std::vector<Set>* extra;
  int size() const { return (int)base->size() + (int)extra->size(); }
  const Set& get(int i) const { return i < (int)base->size() ? (*base)[i] : (*extra)[i - (int)base->size()]; }
};

struct Earley {
  const Grammar& g;
  explicit Earley(const Grammar& gr) : g(gr) {}

  const Sym* sym_at(const Item& it) const {
    if (it.kind != IT_NORMAL) return nullptr;
    const Alt& alt = g.alts[it.a];
    return it.b < (int)alt.syms.size() ? &alt.syms[it.b] : nullptr;
  }

  // predict and complete until nothing changes; `cur` is set number `i` of the view
  void closure(const View& v, Set& cur, int i) const {
    bool changed = true;
    while (changed) {
      changed = false;
      for (size_t k = 0; k < cur.size(); ++k) {
        Item it = cur[k];
        if (it.kind == IT_NORMAL) {
          const Sym* s = sym_at(it);
          if (s) {
            if (s->kind == SYM_NT) {
              for (int a : g.rule_alts[s->arg]) changed |= add_item(cur, {IT_NORMAL, a, 0, i, 0});
            } else if (s->kind == SYM_TD) {
              changed |= add_item(cur, {IT_TDFREE, s->arg, 0, i, 0});
            }
          } else {
            changed |= complete_rule(v, cur, i, g.alts[it.a].rule, it.origin);
          }
        } else if (it.kind == IT_TDFREE) {
          if (g.tds[it.a].stops.empty()) changed |= complete_td(v, cur, i, it.a, it.origin);
        } else if (it.kind == IT_TDDONE) {
          changed |= complete_td(v, cur, i, it.a, it.origin);
        } else {   // TDWAIT: the tag's sub-grammar starts here
          const TagDispatch& td = g.tds[it.a];
          for (int a : g.rule_alts[td.tag_rule[it.b]]) changed |= add_item(cur, {IT_NORMAL, a, 0, i, 0});
        }
      }
    }
  }
  bool complete_rule(const View& v, Set& cur, int i, int rule, int origin) const {
    bool changed = false;
    const Set& os = origin == i ? cur : v.get(origin);
    for (size_t q = 0; q < os.size(); ++q) {
      Item p = os[q];
      if (p.kind == IT_NORMAL) {
        const Sym* s = sym_at(p);
        if (s && s->kind == SYM_NT && s->arg == rule && p.aux == 0)
          changed |= add_item(cur, {IT_NORMAL, p.a, p.b + 1, p.origin, 0});
      } else if (p.kind == IT_TDWAIT) {
        if (g.tds[p.a].tag_rule[p.b] == rule) changed |= add_item(cur, {IT_TDFREE, p.a, 0, p.origin, 0});
      }
    }
    return changed;
  }
  bool complete_td(const View& v, Set& cur, int i, int td, int origin) const {
    bool changed = false;
    const Set& os = origin == i ? cur : v.get(origin);
    for (size_t q = 0; q < os.size(); ++q) {
      Item p = os[q];
      const Sym* s = sym_at(p);
      if (s && s->kind == SYM_TD && s->arg == td) changed |= add_item(cur, {IT_NORMAL, p.a, p.b + 1, p.origin, 0});
    }
    return changed;
  }
  static bool ends_with(const std::string& s, const std::string& suf) {
    return s.size() >= suf.size() && s.compare(s.size() - suf.size(), suf.size(), suf) == 0;
  }
  void scan(const Set& cur, Set& next, uint8_t byte) const {
    for (const Item& it : cur) {
      if (it.kind == IT_NORMAL) {
        const Sym* s = sym_at(it);
        if (!s) continue;
        if (s->kind == SYM_BYTE) {
          if (s->arg == (int)byte) add_item(next, {IT_NORMAL, it.a, it.b + 1, it.origin, 0});
        } else if (s->kind == SYM_CPSET) {
          uint32_t na = 0;
          int r = cpset_step(g.cpsets[s->arg], it.aux, byte, &na);
          if (r == 2) add_item(next, {IT_NORMAL, it.a, it.b + 1, it.origin, 0});
          else if (r == 1) add_item(next, {IT_NORMAL, it.a, it.b, it.origin, na});
        }
      } else if (it.kind == IT_TDFREE) {
        const TagDispatch& td = g.tds[it.a];
        std::string text = td.prefixes[it.b];
        text.push_back((char)byte);
        bool matched = false;
        for (size_t j = 0; j < td.tags.size(); ++j) {
          if (ends_with(text, td.tags[j])) {
            matched = true;
            if (!td.tag_dead[j]) add_item(next, {IT_TDWAIT, it.a, (int)j, it.origin, 0});
          }
        }
        if (!matched) {
          for (const std::string& st : td.stops)
            if (ends_with(text, st)) { matched = true; add_item(next, {IT_TDDONE, it.a, 0, it.origin, 0}); break; }
        }
        if (!matched) {   // keep the longest suffix that is still a proper prefix of a tag / stop string
          for (size_t cut = 0; cut <= text.size(); ++cut) {
            auto f = td.prefix_id.find(text.substr(cut));
            if (f != td.prefix_id.end()) { add_item(next, {IT_TDFREE, it.a, f->second, it.origin, 0}); break; }
          }
        }
      }
    }
  }
  Set initial() const {
    Set s;
    for (int a : g.rule_alts[g.root]) add_item(s, {IT_NORMAL, a, 0, 0, 0});
    std::vector<Set> none, none2;
    View v{&none, &none2};
    closure(v, s, 0);
    return s;
  }
  // feed bytes after `base`; on success the new sets are in `extra`
  bool feed(const std::vector<Set>& base, std::vector<Set>& extra, const uint8_t* bytes, int n) const {
    View v{&base, &extra};
    for (int k = 0; k < n; ++k) {
      const Set& cur = v.get(v.size() - 1);
      Set next;
      scan(cur, next, bytes[k]);
      if (next.empty()) return false;
      int idx = v.size();
      closure(v, next, idx);
      extra.push_back(std::move(next));
    }
    return true;
  }
  bool root_complete(const Set& last) const {
    for (const Item& it : last)
      if (it.kind == IT_NORMAL && it.origin == 0 && g.alts[it.a].rule == g.root && it.b == (int)g.alts[it.a].syms.size()) return true;
    return false;
  }
};

struct VocabO {
  std::vector<uint8_t> bytes;
  std::vector<int64_t> offsets;
  int32_t size = 0, eos = -1;
  std::vector<char> special;
};

struct Matcher {
  const Grammar* g;
  Earley e;
  std::vector<Set> chart;
  bool terminated = false;
  explicit Matcher(const Grammar* gr) : g(gr), e(*gr) { chart.push_back(e.initial()); }
};

template <class F>
void parallel_for(int n, int nthreads, F f) {
  if (nthreads <= 1) { f(0, n); return; }
  std::vector<std::thread> th;
  int chunk = (n + nthreads - 1) / nthreads;
  for (int t = 0; t < nthreads; ++t) {
    int lo = t * chunk, hi = std::min(n, lo + chunk);
    if (lo >= hi) break;
    th.emplace_back([=] { f(lo, hi); });
  }
  for (auto& t : th) t.join();
}

// ------------------------------------------------------------------------------------------
// interpreter for exported tables: rules are byte-level automata whose edges are byte classes
// or references to other rules (Section 3.3: "structures are represented as multiple FSMs")
// ------------------------------------------------------------------------------------------

struct Tables {
  int n_rules = 0, n_states = 0, root_rule = 0, root_nullable = 0;
  std::vector<int32_t> rule_start, state_rule;
  std::vector<uint8_t> state_final;
  std::vector<int32_t> cb, cc, ct, rb, rr, rt;
  std::vector<uint32_t> class_bits;
  // counted repetitions (Section 3.6, "the parser state for R{l,r} is (R{l,r}, k)"): rule r with rep_hi[r] != 0 is
  // X{rep_lo[r], rep_hi[r]} on the automaton of X; ci / ri mark the edges that start the next iteration
  std::vector<int32_t> rep_lo, rep_hi;
  std::vector<uint8_t> ci, ri;
  std::map<std::pair<int, int>, std::vector<uint8_t>> cls_cache;     // (state, count) -> per-token class (filled lazily)
  bool class_has(int c, uint8_t b) const { return (class_bits[(size_t)c * 8 + (b >> 5)] >> (b & 31)) & 1u; }
  bool scannable(int s) const { return cb[s + 1] > cb[s]; }
  bool counted(int s) const { return !rep_hi.empty() && rep_hi[state_rule[s]] != 0; }
  // may an item at state s that has finished k iterations start another one?
  bool may_iterate(int s, int k) const { return k + 1 < rep_hi[state_rule[s]]; }
  // is an item at state s with count k a finished instance of its rule?
  bool complete(int s, int k) const { return state_final[s] && (!counted(s) || k + 1 >= rep_lo[state_rule[s]]); }
  bool citer(int e) const { return !ci.empty() && ci[e]; }
  bool riter(int e) const { return !ri.empty() && ri[e]; }
};

// origin -1: the unknown context that referenced the rule.  k: inside a counted repetition, the iterations finished
// before the current one (0 elsewhere).
struct TItem { int state, origin, k; };
typedef std::vector<TItem> TSet;
inline bool tadd(TSet& s, TItem it) {
  for (const TItem& x : s) if (x.state == it.state && x.origin == it.origin && x.k == it.k) return false;
  s.push_back(it);
  return true;
}
struct TView {
  const std::vector<TSet>* base;
  std::vector<TSet>* extra;
  int size() const { return (int)base->size() + (int)extra->size(); }
  const TSet& get(int i) const { return i < (int)base->size() ? (*base)[i] : (*extra)[i - (int)base->size()]; }
};

// predict + complete to a fixpoint.  Completing an item whose origin is the unknown context
// cannot advance anything here; it is reported through *left_rule.
// An edge that starts the next iteration of a counted repetition exists only while k + 1 < hi and leads to k + 1.
void tclosure(const Tables& t, const TView& v, TSet& cur, int i, bool* left_rule) {
  bool changed = true;
  while (changed) {
    changed = false;
    for (size_t k = 0; k < cur.size(); ++k) {
      TItem it = cur[k];
      for (int e = t.rb[it.state]; e < t.rb[it.state + 1]; ++e) {
        if (t.riter(e) && !t.may_iterate(it.state, it.k)) continue;
        changed |= tadd(cur, {t.rule_start[t.rr[e]], i, 0});
      }
      if (t.complete(it.state, it.k)) {
        if (it.origin < 0) { if (left_rule) *left_rule = true; continue; }
        int rule = t.state_rule[it.state];
        const TSet& os = it.origin == i ? cur : v.get(it.origin);
        for (size_t q = 0; q < os.size(); ++q) {
          TItem p = os[q];
          for (int e = t.rb[p.state]; e < t.rb[p.state + 1]; ++e) {
            if (t.rr[e] != rule) continue;
            if (t.riter(e)) { if (t.may_iterate(p.state, p.k)) changed |= tadd(cur, {t.rt[e], p.origin, p.k + 1}); }
            else changed |= tadd(cur, {t.rt[e], p.origin, p.k});
          }
        }
      }
    }
  }
}
void tscan(const Tables& t, const TSet& cur, TSet& next, uint8_t b) {
  for (const TItem& it : cur)
    for (int e = t.cb[it.state]; e < t.cb[it.state + 1]; ++e) {
      if (!t.class_has(t.cc[e], b)) continue;
      if (t.citer(e)) { if (t.may_iterate(it.state, it.k)) tadd(next, {t.ct[e], it.origin, it.k + 1}); }
      else tadd(next, {t.ct[e], it.origin, it.k});
    }
}
bool tfeed(const Tables& t, const std::vector<TSet>& base, std::vector<TSet>& extra, const uint8_t* bytes, int n) {
  TView v{&base, &extra};
  for (int k = 0; k < n; ++k) {
    TSet next;
    tscan(t, v.get(v.size() - 1), next, bytes[k]);
    if (next.empty()) return false;
    tclosure(t, v, next, v.size(), nullptr);
    extra.push_back(std::move(next));
  }
  return true;
}

// class of one token at one scannable state: 1 accepted, 2 uncertain, 0 rejected.
// The parse starts from the single item (state, unknown context, count); its first byte must be taken
// by one of the state's own byte-class edges.  Accepted: every byte is consumed and the set
// stays non-empty.  Uncertain: not accepted, but the state's rule finished (the parse would
// continue in the unknown context) with bytes left.  Otherwise rejected.
int classify_one(const Tables& t, int state, int count, const uint8_t* bytes, int n) {
  if (n == 0) return 0;
  std::vector<TSet> base(1), extra;
  base[0].push_back({state, -1, count});
  TView v{&base, &extra};
  bool uncertain = false;
  for (int k = 0; k < n; ++k) {
    TSet next;
    tscan(t, v.get(v.size() - 1), next, bytes[k]);
    if (next.empty()) return uncertain ? 2 : 0;
    bool left = false;
    tclosure(t, v, next, v.size(), &left);
    if (left && k + 1 < n) uncertain = true;
    extra.push_back(std::move(next));
  }
  return 1;
}

struct TMatcher {
  const Tables* t;
  std::vector<TSet> chart;
  explicit TMatcher(const Tables* tb) : t(tb) { reset(); }
  void reset() {
    chart.clear();
    TSet s;
    tadd(s, {t->rule_start[t->root_rule], 0, 0});
    std::vector<TSet> none, none2;
    TView v{&none, &none2};
    tclosure(*t, v, s, 0, nullptr);
    chart.push_back(s);
  }
  bool can_terminate() const {
    if (chart.size() == 1 && t->root_nullable) return true;
    for (const TItem& it : chart.back())
      if (it.origin == 0 && t->complete(it.state, it.k) && t->state_rule[it.state] == t->root_rule) return true;
    return false;
  }
};

inline void set_bit(uint32_t* words, int64_t i) { words[i >> 5] |= 1u << (i & 31); }

}  // namespace

// ------------------------------------------------------------------------------------------
// C interface (ctypes)
// ------------------------------------------------------------------------------------------

extern "C" {

void* orc_grammar_create(const char* ebnf, const char* root, char* err, int errlen) {
  try {
    return grammar_from_ebnf(ebnf, root ? root : "root");
  } catch (const std::exception& e) {
    if (err && errlen > 0) { std::strncpy(err, e.what(), errlen - 1); err[errlen - 1] = 0; }
    return nullptr;
  }
}
void orc_grammar_destroy(void* g) { delete (Grammar*)g; }
int orc_grammar_num_rules(void* g) { return (int)((Grammar*)g)->names.size(); }

void* orc_vocab_create(const uint8_t* bytes, const int64_t* offsets, int32_t size, int32_t eos,
                       const int32_t* special, int32_t n_special) {
  VocabO* v = new VocabO();
  v->size = size; v->eos = eos;
  v->offsets.assign(offsets, offsets + size + 1);
  v->bytes.assign(bytes, bytes + offsets[size]);
  v->special.assign(size, 0);
  for (int i = 0; i < n_special; ++i) v->special[special[i]] = 1;
  return v;
}
void orc_vocab_destroy(void* v) { delete (VocabO*)v; }

void* orc_matcher_create(void* g) { return new Matcher((Grammar*)g); }
void orc_matcher_destroy(void* m) { delete (Matcher*)m; }
void orc_matcher_reset(void* mp) {
  Matcher* m = (Matcher*)mp;
  m->chart.clear();
  m->chart.push_back(m->e.initial());
  m->terminated = false;
}
int orc_matcher_num_sets(void* m) { return (int)((Matcher*)m)->chart.size(); }
int orc_matcher_set_size(void* m, int i) { return (int)((Matcher*)m)->chart[i].size(); }
int orc_matcher_is_terminated(void* m) { return ((Matcher*)m)->terminated ? 1 : 0; }

// 1 = accepted (chart advanced); 0 = refused (chart unchanged)
int orc_matcher_accept_bytes(void* mp, const uint8_t* bytes, int n) {
  Matcher* m = (Matcher*)mp;
  if (m->terminated) return 0;
  std::vector<Set> extra;
  if (!m->e.feed(m->chart, extra, bytes, n)) return 0;
  for (auto& s : extra) m->chart.push_back(std::move(s));
  return 1;
}
int orc_matcher_can_terminate(void* mp) {
  Matcher* m = (Matcher*)mp;
  return m->e.root_complete(m->chart.back()) ? 1 : 0;
}
// 1 = accepted; 0 = refused (state unchanged); 2 = EOS accepted, matcher terminated
int orc_matcher_accept_token(void* mp, void* vp, int32_t token) {
  Matcher* m = (Matcher*)mp;
  VocabO* v = (VocabO*)vp;
  if (m->terminated || token < 0 || token >= v->size) return 0;
  if (token == v->eos) {
    if (!m->e.root_complete(m->chart.back())) return 0;
    m->terminated = true;
    return 2;
  }
  int n = (int)(v->offsets[token + 1] - v->offsets[token]);
  if (v->special[token] || n == 0) return 0;
  return orc_matcher_accept_bytes(mp, v->bytes.data() + v->offsets[token], n);
}
// words: ceil(V/32) uint32, bit j of word w = token 32w+j, 1 = allowed
void orc_matcher_mask(void* mp, void* vp, uint32_t* words, int nthreads) {
  Matcher* m = (Matcher*)mp;
  VocabO* v = (VocabO*)vp;
  int nwords = (v->size + 31) / 32;
  std::memset(words, 0, sizeof(uint32_t) * nwords);
  if (m->terminated) return;
  parallel_for(nwords, nthreads, [&](int wlo, int whi) {
    std::vector<Set> extra;
    for (int w = wlo; w < whi; ++w) {
      for (int j = 0; j < 32; ++j) {
        int tok = w * 32 + j;
        if (tok >= v->size) break;
        bool ok;
        if (tok == v->eos) ok = m->e.root_complete(m->chart.back());
        else {
          int n = (int)(v->offsets[tok + 1] - v->offsets[tok]);
          if (v->special[tok] || n == 0) ok = false;
          else { extra.clear(); ok = m->e.feed(m->chart, extra, v->bytes.data() + v->offsets[tok], n); }
        }
        if (ok) words[w] |= 1u << j;
      }
    }
  });
}

// logits[r][c] = -inf where bit (r, c) is 0; other elements untouched
void orc_apply_f32(float* logits, int32_t rows, int32_t vocab, int64_t row_stride, const uint32_t* mask, int64_t mask_stride) {
  const uint32_t ninf = 0xFF800000u;
  for (int32_t r = 0; r < rows; ++r)
    for (int32_t c = 0; c < vocab; ++c)
      if (!((mask[r * mask_stride + (c >> 5)] >> (c & 31)) & 1u)) std::memcpy(&logits[r * row_stride + c], &ninf, 4);
}
void orc_apply_bf16(uint16_t* logits, int32_t rows, int32_t vocab, int64_t row_stride, const uint32_t* mask, int64_t mask_stride) {
  for (int32_t r = 0; r < rows; ++r)
    for (int32_t c = 0; c < vocab; ++c)
      if (!((mask[r * mask_stride + (c >> 5)] >> (c & 31)) & 1u)) logits[r * row_stride + c] = 0xFF80u;
}

// ---- exported-table side -----------------------------------------------------------------

void* orc_tables_create(int32_t n_rules, int32_t n_states, int32_t n_classes, int32_t root_rule, int32_t root_nullable,
                        const int32_t* rule_start, const int32_t* state_rule, const uint8_t* state_final,
                        const int32_t* cedge_begin, const int32_t* cedge_class, const int32_t* cedge_target,
                        const int32_t* redge_begin, const int32_t* redge_rule, const int32_t* redge_target,
                        const uint32_t* class_bits, const int32_t* rule_rep_lo, const int32_t* rule_rep_hi,
                        const uint8_t* cedge_iter, const uint8_t* redge_iter) {
  Tables* t = new Tables();
  t->n_rules = n_rules; t->n_states = n_states; t->root_rule = root_rule; t->root_nullable = root_nullable;
  t->rule_start.assign(rule_start, rule_start + n_rules);
  t->state_rule.assign(state_rule, state_rule + n_states);
  t->state_final.assign(state_final, state_final + n_states);
  t->cb.assign(cedge_begin, cedge_begin + n_states + 1);
  t->cc.assign(cedge_class, cedge_class + t->cb[n_states]);
  t->ct.assign(cedge_target, cedge_target + t->cb[n_states]);
  t->rb.assign(redge_begin, redge_begin + n_states + 1);
  t->rr.assign(redge_rule, redge_rule + t->rb[n_states]);
  t->rt.assign(redge_target, redge_target + t->rb[n_states]);
  t->class_bits.assign(class_bits, class_bits + (size_t)n_classes * 8);
  if (rule_rep_hi) {        // (all four or none)
    t->rep_lo.assign(rule_rep_lo, rule_rep_lo + n_rules);
    t->rep_hi.assign(rule_rep_hi, rule_rep_hi + n_rules);
    t->ci.assign(cedge_iter, cedge_iter + t->cb[n_states]);
    t->ri.assign(redge_iter, redge_iter + t->rb[n_states]);
  }
  return t;
}
void orc_tables_destroy(void* t) { delete (Tables*)t; }

// out[token] = 1 accepted / 2 uncertain / 0 rejected for every token (EOS, specials, empty: 0)
// `count`: inside a counted repetition, the iterations finished before the current one (0 elsewhere)
void orc_tables_classify(void* tp, void* vp, int32_t state, int32_t count, uint8_t* out, int nthreads) {
  Tables* t = (Tables*)tp;
  VocabO* v = (VocabO*)vp;
  parallel_for(v->size, nthreads, [&](int lo, int hi) {
    for (int tok = lo; tok < hi; ++tok) {
      int n = (int)(v->offsets[tok + 1] - v->offsets[tok]);
      if (tok == v->eos || v->special[tok] || n == 0) { out[tok] = 0; continue; }
      out[tok] = (uint8_t)classify_one(*t, state, count, v->bytes.data() + v->offsets[tok], n);
    }
  });
}

void* orc_tmatcher_create(void* t) { return new TMatcher((Tables*)t); }
void orc_tmatcher_destroy(void* m) { delete (TMatcher*)m; }
void orc_tmatcher_reset(void* m) { ((TMatcher*)m)->reset(); }
int orc_tmatcher_accept_bytes(void* mp, const uint8_t* bytes, int n) {
  TMatcher* m = (TMatcher*)mp;
  std::vector<TSet> extra;
  if (!tfeed(*m->t, m->chart, extra, bytes, n)) return 0;
  for (auto& s : extra) m->chart.push_back(std::move(s));
  return 1;
}
int orc_tmatcher_can_terminate(void* m) { return ((TMatcher*)m)->can_terminate() ? 1 : 0; }
int orc_tmatcher_num_sets(void* m) { return (int)((TMatcher*)m)->chart.size(); }
// items of set i as (state, origin) pairs; returns the count
int orc_tmatcher_get_set(void* mp, int i, int32_t* out, int cap) {
  TMatcher* m = (TMatcher*)mp;
  const TSet& s = m->chart[i];
  for (size_t k = 0; k < s.size() && (int)k < cap; ++k) { out[2 * k] = s[k].state; out[2 * k + 1] = s[k].origin; }
  return (int)s.size();
}
// the iteration counts of the items of set i, in the same order
int orc_tmatcher_get_set_counts(void* mp, int i, int32_t* out, int cap) {
  TMatcher* m = (TMatcher*)mp;
  const TSet& s = m->chart[i];
  for (size_t k = 0; k < s.size() && (int)k < cap; ++k) out[k] = s[k].k;
  return (int)s.size();
}
// plain definition on the tables: allowed iff every byte leaves a non-empty set
void orc_tmatcher_mask_plain(void* mp, void* vp, uint32_t* words, int nthreads) {
  TMatcher* m = (TMatcher*)mp;
  VocabO* v = (VocabO*)vp;
  int nwords = (v->size + 31) / 32;
  std::memset(words, 0, sizeof(uint32_t) * nwords);
  parallel_for(nwords, nthreads, [&](int wlo, int whi) {
    std::vector<TSet> extra;
    for (int w = wlo; w < whi; ++w)
      for (int j = 0; j < 32; ++j) {
        int tok = w * 32 + j;
        if (tok >= v->size) break;
        bool ok;
        int n = (int)(v->offsets[tok + 1] - v->offsets[tok]);
        if (tok == v->eos) ok = m->can_terminate();
        else if (v->special[tok] || n == 0) ok = false;
        else { extra.clear(); ok = tfeed(*m->t, m->chart, extra, v->bytes.data() + v->offsets[tok], n); }
        if (ok) words[w] |= 1u << j;
      }
  });
}
// the run-time merge rule: collect the scannable states of the current set; a token accepted by
// at least one state's cache is allowed; otherwise, if some state's cache calls it uncertain, it
// is checked against the whole chart; otherwise it is rejected.  n_checked counts full checks.
void orc_tmatcher_mask_merged(void* mp, void* vp, uint32_t* words, int64_t* n_checked) {
  TMatcher* m = (TMatcher*)mp;
  Tables* t = const_cast<Tables*>(m->t);
  VocabO* v = (VocabO*)vp;
  int nwords = (v->size + 31) / 32;
  std::memset(words, 0, sizeof(uint32_t) * nwords);
  std::vector<std::pair<int, int>> states;          // (state, count)
  for (const TItem& it : m->chart.back())
    if (t->scannable(it.state) && std::find(states.begin(), states.end(), std::make_pair(it.state, it.k)) == states.end()) states.push_back({it.state, it.k});
  for (auto s : states)
    if (!t->cls_cache.count(s)) {
      std::vector<uint8_t> cls(v->size);
      orc_tables_classify(t, v, s.first, s.second, cls.data(), 1);
      t->cls_cache[s] = cls;
    }
  int64_t checked = 0;
  std::vector<TSet> extra;
  for (int tok = 0; tok < v->size; ++tok) {
    int n = (int)(v->offsets[tok + 1] - v->offsets[tok]);
    if (tok == v->eos) { if (m->can_terminate()) set_bit(words, tok); continue; }
    if (v->special[tok] || n == 0) continue;
    bool acc = false, unc = false;
    for (auto s : states) { uint8_t c = t->cls_cache[s][tok]; acc |= c == 1; unc |= c == 2; }
    if (!acc && unc) { ++checked; extra.clear(); acc = tfeed(*t, m->chart, extra, v->bytes.data() + v->offsets[tok], n); }
    if (acc) set_bit(words, tok);
  }
  if (n_checked) *n_checked = checked;
}

}  // extern "C"
