// Host front end (see frontend.h).  Pipeline:
//   text --lex/parse--> expression trees --Thompson--> NFAs with epsilon and rule-reference edges
//   --bypass nullable references, drop epsilon--> NFAs --subset construction + partition
//   refinement--> one DFA per rule --inline small rules--> --trim--> flat tables + closure lists.
#include "frontend.h"

#include <algorithm>
#include <array>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <map>
#include <memory>
#include <set>
#include <unordered_map>

#include "xg.h"

namespace xg {
namespace {

[[noreturn]] void fail(int status, const std::string& msg) { throw FrontendError{status, msg}; }

// ------------------------------------------------------------------------------------------
// byte sets
// ------------------------------------------------------------------------------------------
struct ByteSet {
  std::array<uint32_t, 8> w{};
  void set(int b) { w[b >> 5] |= 1u << (b & 31); }
  void set_range(int lo, int hi) { for (int b = lo; b <= hi; ++b) set(b); }
  bool has(int b) const { return (w[b >> 5] >> (b & 31)) & 1u; }
  bool empty() const { for (uint32_t x : w) if (x) return false; return true; }
  void merge(const ByteSet& o) { for (int i = 0; i < 8; ++i) w[i] |= o.w[i]; }
  bool operator==(const ByteSet& o) const { return w == o.w; }
  bool operator<(const ByteSet& o) const { return w < o.w; }
};

// ------------------------------------------------------------------------------------------
// expression trees
// ------------------------------------------------------------------------------------------
struct TagSpec {
  std::vector<std::string> tags;
  std::vector<std::string> tag_rules;
  std::vector<std::string> stops;
};
struct Expr;
typedef std::shared_ptr<Expr> ExprP;
struct Expr {
  enum Kind { kBytes, kClass, kRef, kSeq, kAlt, kRepeat, kTagDispatch } kind;
  std::string bytes;                                  // kBytes
  std::vector<std::pair<uint32_t, uint32_t>> ranges;  // kClass: code-point ranges (sorted, disjoint)
  std::string name;                                   // kRef
  std::vector<ExprP> kids;                            // kSeq, kAlt, kRepeat (one child)
  int lo = 0, hi = 0;                                 // kRepeat: hi < 0 means unbounded
  TagSpec tag;                                        // kTagDispatch
};
ExprP make(Expr::Kind k) { auto e = std::make_shared<Expr>(); e->kind = k; return e; }

void put_utf8(std::string& out, uint32_t cp) {
  if (cp <= 0x7F) { out += (char)cp; return; }
  if (cp <= 0x7FF) { out += (char)(0xC0 | (cp >> 6)); out += (char)(0x80 | (cp & 63)); return; }
  if (cp <= 0xFFFF) { out += (char)(0xE0 | (cp >> 12)); out += (char)(0x80 | ((cp >> 6) & 63)); out += (char)(0x80 | (cp & 63)); return; }
  out += (char)(0xF0 | (cp >> 18)); out += (char)(0x80 | ((cp >> 12) & 63)); out += (char)(0x80 | ((cp >> 6) & 63)); out += (char)(0x80 | (cp & 63));
}

// ------------------------------------------------------------------------------------------
// lexer + parser for the grammar text
// ------------------------------------------------------------------------------------------
struct Token {
  enum Type { kEnd, kIdent, kDefine, kString, kClass, kBar, kLParen, kRParen, kStar, kPlus, kQuestion, kLBrace, kRBrace, kComma, kInt, kEquals } type = kEnd;
  std::string text;                                   // identifier / decoded string bytes
  std::vector<std::pair<uint32_t, uint32_t>> ranges;  // class
  int value = 0;
  size_t offset = 0;
};

class Lexer {
 public:
  explicit Lexer(const std::string& src) : src_(src) {}
  std::vector<Token> run() {
    std::vector<Token> out;
    while (true) {
      skip_space();
      Token t;
      t.offset = i_;
      if (i_ >= src_.size()) { t.type = Token::kEnd; out.push_back(t); break; }
      unsigned char c = src_[i_];
      if (isalpha(c) || c == '_') {
        size_t j = i_;
        while (j < src_.size() && (isalnum((unsigned char)src_[j]) || src_[j] == '_')) ++j;
        t.type = Token::kIdent; t.text = src_.substr(i_, j - i_); i_ = j;
      } else if (isdigit(c)) {
        long v = 0;
        while (i_ < src_.size() && isdigit((unsigned char)src_[i_])) { v = v * 10 + (src_[i_++] - '0'); if (v > 1000000) err("number too large"); }
        t.type = Token::kInt; t.value = (int)v;
      } else if (c == ':' && src_.compare(i_, 3, "::=") == 0) { t.type = Token::kDefine; i_ += 3; }
      else if (c == '"') { t.type = Token::kString; t.text = read_string(); }
      else if (c == '[') { t.type = Token::kClass; t.ranges = read_class(); }
      else {
        ++i_;
        switch (c) {
          case '|': t.type = Token::kBar; break;
          case '(': t.type = Token::kLParen; break;
          case ')': t.type = Token::kRParen; break;
          case '*': t.type = Token::kStar; break;
          case '+': t.type = Token::kPlus; break;
          case '?': t.type = Token::kQuestion; break;
          case '{': t.type = Token::kLBrace; break;
          case '}': t.type = Token::kRBrace; break;
          case ',': t.type = Token::kComma; break;
          case '=': t.type = Token::kEquals; break;
          default: --i_; err(std::string("unexpected character '") + (char)c + "'");
        }
      }
      out.push_back(t);
    }
    return out;
  }

 private:
  const std::string& src_;
  size_t i_ = 0;
  [[noreturn]] void err(const std::string& m) { fail(XG_ERR_PARSE, "grammar text: " + m + " at offset " + std::to_string(i_)); }
  void skip_space() {
    while (i_ < src_.size()) {
      char c = src_[i_];
      if (c == '#') { while (i_ < src_.size() && src_[i_] != '\n') ++i_; }
      else if (c == ' ' || c == '\t' || c == '\r' || c == '\n') ++i_;
      else break;
    }
  }
  uint32_t read_hex(int digits) {
    uint32_t v = 0;
    for (int k = 0; k < digits; ++k) {
      if (i_ >= src_.size() || !isxdigit((unsigned char)src_[i_])) err("bad hexadecimal escape");
      char c = src_[i_++];
      v = v * 16 + (uint32_t)(isdigit((unsigned char)c) ? c - '0' : (tolower(c) - 'a' + 10));
    }
    return v;
  }
  // one (possibly escaped) unit; sets *raw_byte when it is \xHH outside a class
  uint32_t read_unit(bool in_class, bool* raw_byte) {
    *raw_byte = false;
    unsigned char c = src_[i_];
    if (c != '\\') {
      ++i_;
      if (c < 0x80) return c;
      int extra = c >= 0xF0 ? 3 : c >= 0xE0 ? 2 : c >= 0xC0 ? 1 : -1;
      if (extra < 0) err("invalid UTF-8 in grammar text");
      uint32_t cp = c & (0xFF >> (extra + 2));
      for (int k = 0; k < extra; ++k) {
        if (i_ >= src_.size() || ((unsigned char)src_[i_] & 0xC0) != 0x80) err("invalid UTF-8 in grammar text");
        cp = (cp << 6) | ((unsigned char)src_[i_++] & 63);
      }
      return cp;
    }
    ++i_;
    if (i_ >= src_.size()) err("dangling backslash");
    char e = src_[i_++];
    switch (e) {
      case 'n': return 10; case 't': return 9; case 'r': return 13;
      case '\\': case '"': case '\'': case '/': return (uint32_t)e;
      case 'x': *raw_byte = !in_class; return read_hex(2);
      case 'u': return read_hex(4);
      case 'U': return read_hex(8);
      default:
        if (in_class && (e == ']' || e == '-' || e == '^')) return (uint32_t)e;
        err(std::string("unknown escape \\") + e);
    }
  }
  std::string read_string() {
    ++i_;
    std::string out;
    while (true) {
      if (i_ >= src_.size()) err("unterminated string literal");
      if (src_[i_] == '"') { ++i_; return out; }
      bool raw;
      uint32_t u = read_unit(false, &raw);
      if (raw) out += (char)u;
      else { if (u > 0x10FFFF || (u >= 0xD800 && u <= 0xDFFF)) err("escape is not a scalar value"); put_utf8(out, u); }
    }
  }
  std::vector<std::pair<uint32_t, uint32_t>> read_class() {
    ++i_;
    bool negate = false;
    if (i_ < src_.size() && src_[i_] == '^') { negate = true; ++i_; }
    std::vector<std::pair<uint32_t, uint32_t>> rs;
    while (true) {
      if (i_ >= src_.size()) err("unterminated character class");
      if (src_[i_] == ']') { ++i_; break; }
      bool raw;
      uint32_t a = read_unit(true, &raw), b = a;
      if (i_ + 1 < src_.size() && src_[i_] == '-' && src_[i_ + 1] != ']') {
        ++i_;
        b = read_unit(true, &raw);
        if (b < a) err("character class range is reversed");
      }
      rs.emplace_back(a, b);
    }
    std::sort(rs.begin(), rs.end());
    std::vector<std::pair<uint32_t, uint32_t>> norm;
    for (auto& r : rs) {
      if (!norm.empty() && r.first <= norm.back().second + 1) norm.back().second = std::max(norm.back().second, r.second);
      else norm.push_back(r);
    }
    if (!negate) return norm;
    std::vector<std::pair<uint32_t, uint32_t>> comp;
    uint32_t from = 0;
    for (auto& r : norm) { if (r.first > from) comp.emplace_back(from, r.first - 1); from = r.second + 1; }
    if (from <= 0x10FFFF) comp.emplace_back(from, 0x10FFFFu);
    return comp;
  }
};

class GrammarParser {
 public:
  explicit GrammarParser(std::vector<Token> toks) : t_(std::move(toks)) {}
  std::vector<std::pair<std::string, ExprP>> run() {
    std::vector<std::pair<std::string, ExprP>> rules;
    while (peek().type != Token::kEnd) {
      if (!starts_rule()) err("expected `name ::=`");
      std::string name = t_[p_].text;
      p_ += 2;
      rules.emplace_back(name, alternatives());
    }
    if (rules.empty()) fail(XG_ERR_PARSE, "grammar text: no rules");
    return rules;
  }

 private:
  std::vector<Token> t_;
  size_t p_ = 0;
  const Token& peek() const { return t_[p_]; }
  const Token& peek2() const { return t_[std::min(p_ + 1, t_.size() - 1)]; }
  [[noreturn]] void err(const std::string& m) { fail(XG_ERR_PARSE, "grammar text: " + m + " at offset " + std::to_string(peek().offset)); }
  void want(Token::Type ty, const char* what) { if (peek().type != ty) err(std::string("expected ") + what); ++p_; }
  bool starts_rule() const { return peek().type == Token::kIdent && peek2().type == Token::kDefine; }

  int depth_ = 0;
  ExprP alternatives() {
    struct Guard { int& d; explicit Guard(int& x) : d(x) { ++d; } ~Guard() { --d; } } guard(depth_);
    if (depth_ > 200) err("expression nested too deeply");
    auto alt = make(Expr::kAlt);
    alt->kids.push_back(sequence());
    while (peek().type == Token::kBar) { ++p_; alt->kids.push_back(sequence()); }
    return alt->kids.size() == 1 ? alt->kids[0] : alt;
  }
  ExprP sequence() {
    auto seq = make(Expr::kSeq);
    while (true) {
      Token::Type ty = peek().type;
      if (ty == Token::kEnd || ty == Token::kBar || ty == Token::kRParen || starts_rule()) break;
      seq->kids.push_back(postfix(primary()));
    }
    return seq;
  }
  ExprP primary() {
    const Token& tk = peek();
    if (tk.type == Token::kString) { auto e = make(Expr::kBytes); e->bytes = tk.text; ++p_; return e; }
    if (tk.type == Token::kClass) { auto e = make(Expr::kClass); e->ranges = tk.ranges; ++p_; return e; }
    if (tk.type == Token::kLParen) { ++p_; auto e = alternatives(); want(Token::kRParen, "')'"); return e; }
    if (tk.type == Token::kIdent) {
      if (tk.text == "TagDispatch" && peek2().type == Token::kLParen) { p_ += 2; return tag_dispatch(); }
      auto e = make(Expr::kRef); e->name = tk.text; ++p_; return e;
    }
    err("expected a literal, class, rule name or '('");
  }
  ExprP postfix(ExprP e) {
    while (true) {
      Token::Type ty = peek().type;
      int lo, hi;
      if (ty == Token::kStar) { lo = 0; hi = -1; ++p_; }
      else if (ty == Token::kPlus) { lo = 1; hi = -1; ++p_; }
      else if (ty == Token::kQuestion) { lo = 0; hi = 1; ++p_; }
      else if (ty == Token::kLBrace) {
        ++p_;
        if (peek().type != Token::kInt) err("expected a repetition count");
        lo = hi = peek().value; ++p_;
        if (peek().type == Token::kComma) {
          ++p_;
          if (peek().type == Token::kInt) { hi = peek().value; ++p_; } else hi = -1;
        }
        want(Token::kRBrace, "'}'");
        if (hi >= 0 && hi < lo) err("repetition bounds are reversed");
      } else break;
      auto rep = make(Expr::kRepeat);
      rep->lo = lo; rep->hi = hi; rep->kids.push_back(e);
      e = rep;
    }
    return e;
  }
  std::vector<std::string> string_list() {
    std::vector<std::string> out;
    want(Token::kLParen, "'('");
    while (peek().type != Token::kRParen) {
      if (peek().type != Token::kString) err("expected a string");
      out.push_back(peek().text); ++p_;
      if (peek().type == Token::kComma) ++p_;
    }
    ++p_;
    return out;
  }
  ExprP tag_dispatch() {       // after `TagDispatch(`
    auto e = make(Expr::kTagDispatch);
    while (peek().type != Token::kRParen) {
      if (peek().type == Token::kLParen) {
        ++p_;
        if (peek().type != Token::kString || peek().text.empty()) err("expected a non-empty tag string");
        e->tag.tags.push_back(peek().text); ++p_;
        want(Token::kComma, "','");
        if (peek().type != Token::kIdent) err("expected a rule name");
        e->tag.tag_rules.push_back(peek().text); ++p_;
        want(Token::kRParen, "')'");
      } else if (peek().type == Token::kIdent && peek().text == "stop_strs") {
        ++p_;
        want(Token::kEquals, "'='");
        e->tag.stops = string_list();
        for (auto& s : e->tag.stops) if (s.empty()) err("empty stop string");
      } else err("expected (\"tag\", rule) or stop_strs=(...)");
      if (peek().type == Token::kComma) ++p_;
    }
    ++p_;
    if (e->tag.tags.empty() && e->tag.stops.empty()) err("TagDispatch needs at least one tag or stop string");
    return e;
  }
};

// ------------------------------------------------------------------------------------------
// automata
// ------------------------------------------------------------------------------------------
struct Edge {
  enum Kind : uint8_t { kEps, kBytes, kRef } kind;
  int rule;        // kRef
  int to;
  ByteSet set;     // kBytes
  bool iter = false;   // inside a counted repetition: the edge starts the next iteration
};
struct Fsm {
  std::vector<std::vector<Edge>> out;
  std::vector<char> fin;
  int start = 0;
  bool has_tag_dispatch = false;
  int add() { out.emplace_back(); fin.push_back(0); return (int)out.size() - 1; }
  int size() const { return (int)out.size(); }
  void eps(int a, int b) { out[a].push_back({Edge::kEps, -1, b, {}}); }
  void bytes(int a, const ByteSet& s, int b) { out[a].push_back({Edge::kBytes, -1, b, s}); }
  void ref(int a, int rule, int b) { out[a].push_back({Edge::kRef, rule, b, {}}); }
};

// well-formed UTF-8 encodings of a code-point range as sequences of byte ranges
typedef std::vector<std::pair<int, int>> ByteRangeSeq;
void utf8_sequences(uint32_t lo, uint32_t hi, std::vector<ByteRangeSeq>& out) {
  if (lo > hi) return;
  static const uint32_t limits[4] = {0x7F, 0x7FF, 0xFFFF, 0x10FFFF};
  // keep surrogates out
  if (lo <= 0xDFFF && hi >= 0xD800) {
    if (lo < 0xD800) utf8_sequences(lo, 0xD7FF, out);
    if (hi > 0xDFFF) utf8_sequences(0xE000, hi, out);
    return;
  }
  // one encoded length per piece
  for (int k = 0; k < 3; ++k)
    if (lo <= limits[k] && hi > limits[k]) { utf8_sequences(lo, limits[k], out); utf8_sequences(limits[k] + 1, hi, out); return; }
  if (hi <= 0x7F) { out.push_back({{(int)lo, (int)hi}}); return; }
  int n = hi <= 0x7FF ? 2 : hi <= 0xFFFF ? 3 : 4;
  // split until the low 6*k bits span a full block wherever the higher bits differ
  for (int k = 1; k < n; ++k) {
    uint32_t m = (1u << (6 * k)) - 1;
    if ((lo & ~m) != (hi & ~m)) {
      if ((lo & m) != 0) { utf8_sequences(lo, lo | m, out); utf8_sequences((lo | m) + 1, hi, out); return; }
      if ((hi & m) != m) { utf8_sequences(lo, (hi & ~m) - 1, out); utf8_sequences(hi & ~m, hi, out); return; }
    }
  }
  std::string a, b;
  put_utf8(a, lo); put_utf8(b, hi);
  ByteRangeSeq seq;
  for (int k = 0; k < n; ++k) seq.emplace_back((unsigned char)a[k], (unsigned char)b[k]);
  out.push_back(seq);
}

// Aho-Corasick automaton over tags and stop strings (Section 3.2)
struct AhoCorasick {
  std::vector<std::array<int, 256>> next;   // goto function completed with failure links
  std::vector<std::vector<int>> ends;       // patterns ending at the node (own or via suffix links)
  explicit AhoCorasick(const std::vector<std::string>& patterns) {
    std::vector<std::array<int, 256>> child;
    std::vector<int> link;
    auto node = [&]() { std::array<int, 256> a; a.fill(-1); child.push_back(a); ends.emplace_back(); link.push_back(0); return (int)child.size() - 1; };
    node();
    for (size_t p = 0; p < patterns.size(); ++p) {
      int u = 0;
      for (unsigned char c : patterns[p]) { if (child[u][c] < 0) { int v = node(); child[u][c] = v; } u = child[u][c]; }
      ends[u].push_back((int)p);
    }
    next.assign(child.size(), {});
    std::vector<int> queue;
    for (int c = 0; c < 256; ++c) {
      int v = child[0][c];
      if (v < 0) next[0][c] = 0; else { next[0][c] = v; link[v] = 0; queue.push_back(v); }
    }
    for (size_t q = 0; q < queue.size(); ++q) {
      int u = queue[q];
      for (int p : ends[link[u]]) ends[u].push_back(p);
      for (int c = 0; c < 256; ++c) {
        int v = child[u][c];
        if (v < 0) next[u][c] = next[link[u]][c];
        else { next[u][c] = v; link[v] = next[link[u]][c]; queue.push_back(v); }
      }
    }
  }
};

constexpr int kKeepDispatchedRules = 8;

// A counted repetition (Section 3.6): rule `rep` stands for body{lo,hi}.  Until the tables are written its automaton
// is a single reference to `body`, so that nullability, trimming and the reference graph see it as an ordinary rule.
struct CountedRule {
  int body = -1, lo = 0, hi = 0;
};

struct Builder {
  std::set<int> keep_as_rule;             // rules that inlining leaves alone
  std::vector<std::string> names;
  std::map<std::string, int> ids;
  std::vector<Fsm> rules;
  int repeat_threshold = 0;               // bounded repetitions with at least this many iterations become counted rules (0: never)
  int max_expanded = 0;                   // the largest bound among the repetitions expanded into explicit states
  std::map<int, CountedRule> counted;     // rule id -> what it repeats
  std::map<int, Fsm> pending;             // automata of the rules made while another rule is being built (appended afterwards)

  int new_rule(const std::string& name) {
    const int id = (int)names.size();
    names.push_back(name);
    ids[name] = id;
    keep_as_rule.insert(id);
    return id;
  }

  int lookup(const std::string& n) const {
    auto it = ids.find(n);
    if (it == ids.end()) fail(XG_ERR_PARSE, "grammar text: undefined rule " + n);
    return it->second;
  }
  // Thompson construction: returns (entry, exit) of a fragment inside f
  int max_states = 1 << 20;
  std::pair<int, int> frag(Fsm& f, const Expr& e) {
    if (f.size() > max_states) fail(XG_ERR_CAPACITY, "a rule automaton exceeds max_rule_states");
    switch (e.kind) {
      case Expr::kBytes: {
        int s = f.add(), cur = s;
        for (unsigned char c : e.bytes) { int n = f.add(); ByteSet bs; bs.set(c); f.bytes(cur, bs, n); cur = n; }
        return {s, cur};
      }
      case Expr::kClass: {
        int s = f.add(), t = f.add();
        std::vector<ByteRangeSeq> seqs;
        for (auto& r : e.ranges) utf8_sequences(r.first, std::min<uint32_t>(r.second, 0x10FFFF), seqs);
        for (auto& seq : seqs) {
          int cur = s;
          for (size_t k = 0; k < seq.size(); ++k) {
            int n = k + 1 == seq.size() ? t : f.add();
            ByteSet bs; bs.set_range(seq[k].first, seq[k].second);
            f.bytes(cur, bs, n);
            cur = n;
          }
        }
        return {s, t};
      }
      case Expr::kRef: { int s = f.add(), t = f.add(); f.ref(s, lookup(e.name), t); return {s, t}; }
      case Expr::kSeq: {
        int s = f.add(), cur = s;
        for (auto& k : e.kids) { auto p = frag(f, *k); f.eps(cur, p.first); cur = p.second; }
        return {s, cur};
      }
      case Expr::kAlt: {
        int s = f.add(), t = f.add();
        for (auto& k : e.kids) { auto p = frag(f, *k); f.eps(s, p.first); f.eps(p.second, t); }
        return {s, t};
      }
      case Expr::kRepeat: {
        if (repeat_threshold > 0 && e.hi >= repeat_threshold) {
          // X{lo,hi} as a rule of its own with a counter in its items: one copy of X whatever the bounds
          const std::string tag = "%rep" + std::to_string(names.size());
          const int body = new_rule(tag + ".body"), rep = new_rule(tag);
          {
            Fsm bf;
            auto p = frag(bf, *e.kids[0]);
            bf.start = p.first; bf.fin[p.second] = 1;
            pending[body] = std::move(bf);
          }
          Fsm rf;
          const int a = rf.add(), z = rf.add();
          rf.ref(a, body, z);
          rf.start = a; rf.fin[z] = 1;
          if (e.lo == 0) rf.fin[a] = 1;
          pending[rep] = std::move(rf);
          counted[rep] = {body, e.lo, e.hi};
          int s = f.add(), t = f.add();
          f.ref(s, rep, t);
          return {s, t};
        }
        max_expanded = std::max(max_expanded, e.hi < 0 ? e.lo : e.hi);
        int s = f.add(), cur = s;
        for (int i = 0; i < e.lo; ++i) { auto p = frag(f, *e.kids[0]); f.eps(cur, p.first); cur = p.second; }
        int t = f.add();
        if (e.hi < 0) {
          int loop = f.add();
          f.eps(cur, loop);
          auto p = frag(f, *e.kids[0]);
          f.eps(loop, p.first); f.eps(p.second, loop); f.eps(loop, t);
        } else {
          for (int i = e.lo; i < e.hi; ++i) { f.eps(cur, t); auto p = frag(f, *e.kids[0]); f.eps(cur, p.first); cur = p.second; }
          f.eps(cur, t);
        }
        return {s, t};
      }
      case Expr::kTagDispatch: return tag_fragment(f, e.tag);
    }
    fail(XG_ERR_INVALID_ARG, "internal: unknown expression kind");
  }
  std::pair<int, int> tag_fragment(Fsm& f, const TagSpec& spec) {
    f.has_tag_dispatch = true;
    std::vector<std::string> patterns = spec.tags;
    patterns.insert(patterns.end(), spec.stops.begin(), spec.stops.end());
    int n_tags = (int)spec.tags.size();
    AhoCorasick ac(patterns);
    int n_nodes = (int)ac.next.size();
    std::vector<int> node_state(n_nodes, -1);
    for (int u = 0; u < n_nodes; ++u) if (ac.ends[u].empty()) node_state[u] = f.add();
    int exit = f.add();
    std::vector<int> dispatch(n_tags, -1);       // state holding the reference edge of tag j
    for (int j = 0; j < n_tags; ++j) { dispatch[j] = f.add(); f.ref(dispatch[j], lookup(spec.tag_rules[j]), node_state[0]); }
    // A dispatch over many tags is a menu of independent structures (one tool each): their rules are kept as
    // rules, so that requests which offer different subsets of a tool pool still share the cache entries of the
    // tools they have in common (Section 3.3; inlined into the dispatching automaton they would be unique to it).
    if (n_tags >= kKeepDispatchedRules) for (int j = 0; j < n_tags; ++j) keep_as_rule.insert(lookup(spec.tag_rules[j]));
    for (int u = 0; u < n_nodes; ++u) {
      if (node_state[u] < 0) continue;
      std::map<int, ByteSet> by_target;          // target state -> bytes
      for (int c = 0; c < 256; ++c) {
        int v = ac.next[u][c];
        if (ac.ends[v].empty()) { by_target[node_state[v]].set(c); continue; }
        bool any_tag = false;
        for (int p : ac.ends[v]) if (p < n_tags) { any_tag = true; by_target[dispatch[p]].set(c); }
        if (!any_tag) by_target[exit].set(c);    // a stop string ends the construct
      }
      for (auto& kv : by_target) f.bytes(node_state[u], kv.second, kv.first);
      if (spec.stops.empty()) f.eps(node_state[u], exit);   // may end anywhere while dispatching
    }
    return {node_state[0], exit};
  }
};

// epsilon closure of every state
std::vector<std::vector<int>> eps_closures(const Fsm& f) {
  int n = f.size();
  std::vector<std::vector<int>> cl(n);
  std::vector<int> mark(n, -1), stack;
  for (int s = 0; s < n; ++s) {
    stack.assign(1, s); mark[s] = s;
    while (!stack.empty()) {
      int u = stack.back(); stack.pop_back();
      cl[s].push_back(u);
      for (const Edge& e : f.out[u]) if (e.kind == Edge::kEps && mark[e.to] != s) { mark[e.to] = s; stack.push_back(e.to); }
    }
  }
  return cl;
}

Fsm drop_epsilon(const Fsm& f) {
  auto cl = eps_closures(f);
  Fsm g;
  g.has_tag_dispatch = f.has_tag_dispatch;
  for (int s = 0; s < f.size(); ++s) g.add();
  g.start = f.start;
  for (int s = 0; s < f.size(); ++s)
    for (int u : cl[s]) {
      if (f.fin[u]) g.fin[s] = 1;
      for (const Edge& e : f.out[u]) if (e.kind != Edge::kEps) g.out[s].push_back(e);
    }
  return g;
}

// subset construction over the alphabet {bytes} + {rule references}; the input has no epsilon edges
Fsm determinize(const Fsm& f, int max_states) {
  Fsm d;
  d.has_tag_dispatch = f.has_tag_dispatch;
  std::map<std::vector<int>, int> index;
  std::vector<int> single(f.size(), -1);              // subsets of one state, the common case
  std::vector<std::vector<int>> subsets;
  auto state_of = [&](std::vector<int>& set) {
    std::sort(set.begin(), set.end());
    set.erase(std::unique(set.begin(), set.end()), set.end());
    if (set.size() == 1) { if (single[set[0]] >= 0) return single[set[0]]; }
    else { auto it = index.find(set); if (it != index.end()) return it->second; }
    int id = d.add();
    if (id >= max_states) fail(XG_ERR_CAPACITY, "a rule automaton exceeds max_rule_states");
    if (set.size() == 1) single[set[0]] = id; else index[set] = id;
    subsets.push_back(set);
    for (int s : set) if (f.fin[s]) d.fin[id] = 1;
    return id;
  };
  std::vector<int> init{f.start};
  d.start = state_of(init);
  for (int cur = 0; cur < (int)subsets.size(); ++cur) {
    std::vector<int> members = subsets[cur];
    std::map<int, std::vector<int>> by_rule;
    std::vector<const Edge*> byte_edges;
    for (int s : members)
      for (const Edge& e : f.out[s]) {
        if (e.kind == Edge::kRef) by_rule[e.rule].push_back(e.to);
        else if (e.kind == Edge::kBytes) byte_edges.push_back(&e);
      }
    for (auto& kv : by_rule) { int t = state_of(kv.second); d.ref(cur, kv.first, t); }
    if (byte_edges.empty()) continue;
    // common case: the byte sets do not overlap, so every edge keeps its single target
    {
      ByteSet seen;
      bool disjoint = true;
      for (const Edge* e : byte_edges) {
        for (int w = 0; w < 8 && disjoint; ++w) disjoint = (seen.w[w] & e->set.w[w]) == 0;
        if (!disjoint) break;
        seen.merge(e->set);
      }
      if (disjoint) {
        std::map<int, ByteSet> by_target;
        for (const Edge* e : byte_edges) by_target[e->to].merge(e->set);
        for (auto& kv : by_target) { std::vector<int> tg{kv.first}; int t = state_of(tg); d.bytes(cur, kv.second, t); }
        continue;
      }
    }
    std::map<std::vector<int>, ByteSet> groups;      // target subset -> bytes
    std::vector<int> targets;
    for (int b = 0; b < 256; ++b) {
      targets.clear();
      for (const Edge* e : byte_edges) if (e->set.has(b)) targets.push_back(e->to);
      if (targets.empty()) continue;
      std::sort(targets.begin(), targets.end());
      targets.erase(std::unique(targets.begin(), targets.end()), targets.end());
      groups[targets].set(b);
    }
    for (auto& kv : groups) { std::vector<int> tg = kv.first; int t = state_of(tg); d.bytes(cur, kv.second, t); }
  }
  return d;
}

// Equal word sequences get equal ids, numbered in order of first appearance.  Open addressing on a
// 64-bit hash of the words; a hit is confirmed against the stored words.
struct SignatureTable {
  std::vector<uint32_t> words;                         // every distinct signature, back to back
  std::vector<std::pair<size_t, size_t>> span;         // id -> (begin, length)
  std::vector<uint64_t> slot_hash;
  std::vector<int> slot_id;                            // -1 = empty
  int size() const { return (int)span.size(); }
  void grow() {
    const size_t cap = slot_id.empty() ? 64 : slot_id.size() * 2;
    std::vector<uint64_t> nh(cap, 0);
    std::vector<int> ni(cap, -1);
    for (size_t k = 0; k < slot_id.size(); ++k) {
      if (slot_id[k] < 0) continue;
      size_t at = (size_t)slot_hash[k] & (cap - 1);
      while (ni[at] >= 0) at = (at + 1) & (cap - 1);
      nh[at] = slot_hash[k]; ni[at] = slot_id[k];
    }
    slot_hash.swap(nh); slot_id.swap(ni);
  }
  int intern(const std::vector<uint32_t>& sig) {
    uint64_t h = 0x9E3779B97F4A7C15ull ^ sig.size();
    for (uint32_t x : sig) { h ^= x; h *= 0xBF58476D1CE4E5B9ull; h ^= h >> 29; }
    if (span.size() * 2 >= slot_id.size()) grow();
    const size_t mask = slot_id.size() - 1;
    size_t at = (size_t)h & mask;
    while (slot_id[at] >= 0) {
      const int id = slot_id[at];
      if (slot_hash[at] == h && span[id].second == sig.size() && std::equal(sig.begin(), sig.end(), words.begin() + span[id].first)) return id;
      at = (at + 1) & mask;
    }
    const int id = (int)span.size();
    span.emplace_back(words.size(), sig.size());
    words.insert(words.end(), sig.begin(), sig.end());
    slot_hash[at] = h; slot_id[at] = id;
    return id;
  }
};

// The outgoing edges of state s with targets replaced by their class: byte sets merged per
// class (ascending class), then the reference edges (ascending rule, class).
struct ClassEdges {
  std::vector<std::pair<int, ByteSet>> bytes;
  std::vector<std::pair<int, int>> refs;
  void collect(const Fsm& f, int s, const std::vector<int>& cls) {
    bytes.clear(); refs.clear();
    for (const Edge& e : f.out[s]) {
      if (e.kind == Edge::kBytes) {
        const int c = cls[e.to];
        size_t k = 0;
        while (k < bytes.size() && bytes[k].first != c) ++k;
        if (k == bytes.size()) bytes.emplace_back(c, e.set); else bytes[k].second.merge(e.set);
      } else refs.emplace_back(e.rule, cls[e.to]);
    }
    std::sort(bytes.begin(), bytes.end(), [](const std::pair<int, ByteSet>& a, const std::pair<int, ByteSet>& b) { return a.first < b.first; });
    std::sort(refs.begin(), refs.end());
  }
  void signature(int head, std::vector<uint32_t>& sig) const {
    sig.clear();
    sig.push_back((uint32_t)head);
    sig.push_back((uint32_t)bytes.size());
    for (auto& b : bytes) { sig.push_back((uint32_t)b.first); sig.insert(sig.end(), b.second.w.begin(), b.second.w.end()); }
    for (auto& r : refs) { sig.push_back((uint32_t)r.first); sig.push_back((uint32_t)r.second); }
  }
};

// the quotient automaton of a partition (classes numbered 0 .. n_cls-1)
Fsm quotient(const Fsm& f, const std::vector<int>& cls, int n_cls) {
  Fsm m;
  m.has_tag_dispatch = f.has_tag_dispatch;
  for (int b = 0; b < n_cls; ++b) m.add();
  std::vector<char> done(n_cls, 0);
  m.start = cls[f.start];
  ClassEdges ce;
  for (int s = 0; s < f.size(); ++s) {
    const int b = cls[s];
    if (f.fin[s]) m.fin[b] = 1;
    if (done[b]) continue;
    done[b] = 1;
    ce.collect(f, s, cls);
    for (const Edge& e : f.out[s]) if (e.kind == Edge::kRef) m.ref(b, e.rule, cls[e.to]);
    for (auto& kv : ce.bytes) m.bytes(b, kv.second, kv.first);
  }
  return m;
}

// Minimisation of an acyclic deterministic automaton in one bottom-up pass: in reverse
// topological order, two states are equivalent iff they agree on acceptance and on their edges
// into already-merged targets.  Returns false (and leaves `out` alone) if the automaton has a cycle.
bool minimize_acyclic(const Fsm& f, Fsm& out) {
  const int n = f.size();
  std::vector<int> indeg(n, 0), order;
  for (int s = 0; s < n; ++s) for (const Edge& e : f.out[s]) ++indeg[e.to];
  for (int s = 0; s < n; ++s) if (!indeg[s]) order.push_back(s);
  for (size_t q = 0; q < order.size(); ++q) for (const Edge& e : f.out[order[q]]) if (--indeg[e.to] == 0) order.push_back(e.to);
  if ((int)order.size() != n) return false;
  SignatureTable table;
  std::vector<int> cls(n, -1);
  ClassEdges ce;
  std::vector<uint32_t> sig;
  for (int k = n - 1; k >= 0; --k) {
    const int s = order[k];
    ce.collect(f, s, cls);
    ce.signature((int)f.fin[s], sig);
    cls[s] = table.intern(sig);
  }
  out = quotient(f, cls, table.size());
  return true;
}

// Merge equivalent states of a deterministic automaton: partition refinement on sparse
// signatures.  A state's signature (its edges with targets replaced by their blocks) is only
// recomputed after one of its targets changed block, and when a block splits the largest part
// keeps the block's id, so a state changes id O(log n) times.
Fsm minimize(const Fsm& f) {
  {
    Fsm quick;
    if (minimize_acyclic(f, quick)) return quick;
  }
  const int n = f.size();
  std::vector<std::vector<int>> pred(n);
  for (int s = 0; s < n; ++s) for (const Edge& e : f.out[s]) pred[e.to].push_back(s);
  std::vector<int> block(n);
  std::vector<std::vector<int>> members;
  {
    int id_of[2] = {-1, -1};
    for (int s = 0; s < n; ++s) {
      int& id = id_of[f.fin[s] ? 1 : 0];
      if (id < 0) { id = (int)members.size(); members.emplace_back(); }
      block[s] = id;
      members[id].push_back(s);
    }
  }
  SignatureTable table;
  std::vector<int> sig_id(n, -1), work(n), touched;
  std::vector<char> queued(n, 1), block_touched;
  for (int s = 0; s < n; ++s) work[s] = s;
  ClassEdges ce;
  std::vector<uint32_t> sig;
  while (!work.empty()) {
    touched.clear();
    block_touched.assign(members.size(), 0);
    for (int s : work) {
      ce.collect(f, s, block);
      ce.signature(0, sig);
      sig_id[s] = table.intern(sig);
      queued[s] = 0;
      if (!block_touched[block[s]]) { block_touched[block[s]] = 1; touched.push_back(block[s]); }
    }
    work.clear();
    for (int b : touched) {
      {
        std::vector<int>& in_place = members[b];
        std::sort(in_place.begin(), in_place.end(), [&](int x, int y) { return sig_id[x] != sig_id[y] ? sig_id[x] < sig_id[y] : x < y; });
        if (sig_id[in_place.front()] == sig_id[in_place.back()]) continue;
      }
      const std::vector<int> mem = members[b];      // a copy: `members` grows below
      size_t best_begin = 0, best_len = 0;                    // the largest part stays
      for (size_t i = 0; i < mem.size();) {
        size_t j = i;
        while (j < mem.size() && sig_id[mem[j]] == sig_id[mem[i]]) ++j;
        if (j - i > best_len) { best_len = j - i; best_begin = i; }
        i = j;
      }
      std::vector<int> stay(mem.begin() + best_begin, mem.begin() + best_begin + best_len);
      for (size_t i = 0; i < mem.size();) {
        size_t j = i;
        while (j < mem.size() && sig_id[mem[j]] == sig_id[mem[i]]) ++j;
        if (i != best_begin) {
          const int id = (int)members.size();
          members.emplace_back(mem.begin() + i, mem.begin() + j);
          for (size_t k = i; k < j; ++k) {
            block[mem[k]] = id;
            for (int p : pred[mem[k]]) if (!queued[p]) { queued[p] = 1; work.push_back(p); }
          }
        }
        i = j;
      }
      members[b] = stay;
    }
  }
  return quotient(f, block, (int)members.size());
}

// breadth-first renumbering from the start state with edges in a fixed order; drops unreachable
// states
Fsm canonical_order(const Fsm& f) {
  std::vector<int> order, id(f.size(), -1);
  order.push_back(f.start); id[f.start] = 0;
  auto sorted_edges = [&](int s) {
    std::vector<const Edge*> es;
    for (const Edge& e : f.out[s]) es.push_back(&e);
    std::stable_sort(es.begin(), es.end(), [](const Edge* a, const Edge* b) {
      if (a->kind != b->kind) return a->kind < b->kind;
      if (a->kind == Edge::kBytes) return a->set < b->set;
      return a->rule < b->rule;
    });
    return es;
  };
  for (size_t q = 0; q < order.size(); ++q)
    for (const Edge* e : sorted_edges(order[q])) if (id[e->to] < 0) { id[e->to] = (int)order.size(); order.push_back(e->to); }
  Fsm g;
  g.has_tag_dispatch = f.has_tag_dispatch;
  for (size_t k = 0; k < order.size(); ++k) g.add();
  g.start = 0;
  for (size_t k = 0; k < order.size(); ++k) {
    int s = order[k];
    g.fin[k] = f.fin[s];
    for (const Edge* e : sorted_edges(s)) { Edge c = *e; c.to = id[e->to]; g.out[k].push_back(c); }
  }
  return g;
}

Fsm normalize(const Fsm& f, int max_states) { return canonical_order(minimize(determinize(drop_epsilon(f), max_states))); }

struct Compiler {
  Builder b;
  FrontendOptions opt;
  int root = 0;
  bool root_nullable = false;

  int n_rules() const { return (int)b.rules.size(); }

  // rules that derive the empty string: fixpoint over "an accepting state is reachable from the
  // start through epsilon edges and references to nullable rules"
  std::vector<char> nullable_rules() {
    std::vector<char> nullable(n_rules(), 0);
    bool changed = true;
    while (changed) {
      changed = false;
      for (int r = 0; r < n_rules(); ++r) {
        if (nullable[r]) continue;
        const Fsm& f = b.rules[r];
        std::vector<char> seen(f.size(), 0);
        std::vector<int> stack{f.start};
        seen[f.start] = 1;
        bool hit = false;
        while (!stack.empty()) {
          int u = stack.back(); stack.pop_back();
          if (f.fin[u]) { hit = true; break; }
          for (const Edge& e : f.out[u])
            if ((e.kind == Edge::kEps || (e.kind == Edge::kRef && nullable[e.rule])) && !seen[e.to]) { seen[e.to] = 1; stack.push_back(e.to); }
        }
        if (hit) { nullable[r] = 1; changed = true; }
      }
    }
    return nullable;
  }

  void remove_nullability() {
    std::vector<char> nullable = nullable_rules();
    root_nullable = nullable[root];
    // a counted rule loses the empty string like every other rule (its users get the bypass below); with a body
    // that derives the empty string, body{lo,hi} is (body minus empty){0,hi}
    for (auto& kv : b.counted) kv.second.lo = nullable[kv.second.body] ? 1 : std::max(kv.second.lo, 1);
    for (Fsm& f : b.rules)
      for (int s = 0; s < f.size(); ++s) {
        size_t n = f.out[s].size();
        for (size_t k = 0; k < n; ++k)
          if (f.out[s][k].kind == Edge::kRef && nullable[f.out[s][k].rule]) { int to = f.out[s][k].to; f.eps(s, to); }
      }
    for (int r = 0; r < n_rules(); ++r) {
      Fsm g = drop_epsilon(b.rules[r]);
      if (g.fin[g.start]) {          // take the empty string out: a fresh, non-accepting start
        int s = g.add();
        g.out[s] = g.out[g.start];
        g.start = s;
      }
      b.rules[r] = g;
    }
  }

  // Rules that derive at least one string; then: drop references to the others, and every state
  // that cannot reach an accepting state.
  // Returns, per rule, whether anything was removed (an untouched rule keeps its automaton as is).
  std::vector<char> trim() {
    int R = n_rules();
    std::vector<char> touched(R, 0);
    std::vector<char> productive(R, 0);
    auto live_states = [&](const Fsm& f) {
      int n = f.size();
      std::vector<std::vector<int>> rev(n);
      for (int s = 0; s < n; ++s)
        for (const Edge& e : f.out[s]) {
          bool usable = e.kind == Edge::kEps || (e.kind == Edge::kBytes && !e.set.empty()) || (e.kind == Edge::kRef && productive[e.rule]);
          if (usable) rev[e.to].push_back(s);
        }
      std::vector<char> live(n, 0);
      std::vector<int> stack;
      for (int s = 0; s < n; ++s) if (f.fin[s]) { live[s] = 1; stack.push_back(s); }
      while (!stack.empty()) { int u = stack.back(); stack.pop_back(); for (int p : rev[u]) if (!live[p]) { live[p] = 1; stack.push_back(p); } }
      return live;
    };
    bool changed = true;
    while (changed) {
      changed = false;
      for (int r = 0; r < R; ++r) if (!productive[r] && live_states(b.rules[r])[b.rules[r].start]) { productive[r] = 1; changed = true; }
    }
    for (int r = 0; r < R; ++r) {
      Fsm& f = b.rules[r];
      std::vector<char> live = live_states(f);
      live[f.start] = 1;           // the start state stays even if the rule derives nothing
      std::vector<int> id(f.size(), -1);
      Fsm g;
      g.has_tag_dispatch = f.has_tag_dispatch;
      for (int s = 0; s < f.size(); ++s) if (live[s]) id[s] = g.add();
      g.start = id[f.start];
      for (int s = 0; s < f.size(); ++s) {
        if (!live[s]) continue;
        g.fin[id[s]] = f.fin[s];
        for (const Edge& e : f.out[s]) {
          if (!live[e.to]) continue;
          if (e.kind == Edge::kRef && !productive[e.rule]) continue;
          if (e.kind == Edge::kBytes && e.set.empty()) continue;
          Edge c = e; c.to = id[e.to];
          g.out[id[s]].push_back(c);
        }
      }
      size_t edges_before = 0, edges_after = 0;
      for (auto& es : f.out) edges_before += es.size();
      for (auto& es : g.out) edges_after += es.size();
      if (g.size() != f.size() || edges_after != edges_before) { f = g; touched[r] = 1; }
    }
    return touched;
  }

  // Replace references to small rules by a copy of their automaton.  A rule that
  // is referenced from a single place may be larger (inlining it duplicates nothing); this also
  // folds alternatives such as the tool calls of a TagDispatch into one deterministic automaton.
  // A rule used a few times may also be somewhat larger as long as size x uses stays bounded
  // (a character rule repeated by a bounded string must not stay a rule of its own: every
  // multi-byte token would leave it and become context-dependent).
  void inline_small_rules(std::vector<char>& renormalized) {
    renormalized.assign(n_rules(), 0);
    if (opt.inline_max_states <= 0) return;
    const int single_use_max = std::max(64, opt.inline_max_states);
    int R = n_rules();
    std::vector<int> uses(R, 0);
    for (const Fsm& f : b.rules) for (auto& es : f.out) for (const Edge& e : es) if (e.kind == Edge::kRef) ++uses[e.rule];
    std::vector<char> candidate(R, 0), done(R, 0);
    std::function<void(int)> process = [&](int r) {       // callees first
      if (done[r]) return;
      done[r] = 1;          // also guards recursion through cycles
      std::set<int> callees;
      for (auto& es : b.rules[r].out) for (const Edge& e : es) if (e.kind == Edge::kRef) callees.insert(e.rule);
      for (int c : callees) if (c != r) process(c);
      const Fsm& f = b.rules[r];
      bool changed = false;
      Fsm g = f;
      for (int s = 0; s < f.size(); ++s) {
        std::vector<Edge> keep;
        const std::vector<Edge> edges = g.out[s];     // g.out may reallocate while copies are appended
        for (const Edge& e : edges) {
          bool take = e.kind == Edge::kRef && e.rule != r && candidate[e.rule] && !b.counted.count(r) &&
                      (b.rules[e.rule].size() <= opt.inline_max_states || uses[e.rule] == 1 ||
                       b.rules[e.rule].size() * uses[e.rule] <= 16 * opt.inline_max_states) &&
                      g.size() + b.rules[e.rule].size() <= opt.max_rule_states;
          if (take) {
            const Fsm& c = b.rules[e.rule];
            int base = g.size();
            for (int k = 0; k < c.size(); ++k) g.add();
            for (int k = 0; k < c.size(); ++k) {
              for (Edge ce : c.out[k]) { if (ce.kind == Edge::kRef) ++uses[ce.rule]; ce.to += base; g.out[base + k].push_back(ce); }
              if (c.fin[k]) g.eps(base + k, e.to);
            }
            keep.push_back({Edge::kEps, -1, base + c.start, {}});
            g.has_tag_dispatch = g.has_tag_dispatch || c.has_tag_dispatch;
            --uses[e.rule];
            changed = true;
          } else keep.push_back(e);
        }
        g.out[s] = keep;
      }
      if (changed) { b.rules[r] = normalize(g, opt.max_rule_states); renormalized[r] = 1; }
      // A rule on a cycle of references may be copied into its users too: each rule is finished before anything
      // copies it and is copied as it then stands, so the expansion ends; a cycle keeps the rule whose processing
      // began first, which ends up referring to itself (any-JSON: object, member and array fold into value).  One
      // level of nesting is then one rule, not three: a closing bracket completes one rule instead of a cascade,
      // and tokens that run from a string into the punctuation behind it stay inside their rule (Section 3.4: only
      // tokens that leave the rule are context-dependent).
      bool self_reference = false;
      for (auto& es : b.rules[r].out) for (const Edge& e : es) self_reference = self_reference || (e.kind == Edge::kRef && e.rule == r);
      candidate[r] = !self_reference && r != root && b.rules[r].size() <= single_use_max && !b.keep_as_rule.count(r);
    };
    for (int r = 0; r < R; ++r) process(r);
  }

  // the automaton a counted rule runs on: its body's, and at every accepting state copies of the start state's
  // edges that begin the next iteration
  Fsm counted_automaton(const CountedRule& c) const {
    Fsm f = b.rules[c.body];
    const std::vector<Edge> first = f.out[f.start];
    for (int s = 0; s < f.size(); ++s)
      if (f.fin[s]) for (Edge e : first) { e.iter = true; f.out[s].push_back(e); }
    return f;
  }

  FlatGrammar flatten() {
    int R = n_rules();
    std::map<int, Fsm> counted_fsm;
    auto fsm_of = [&](int r) -> const Fsm& {
      auto c = b.counted.find(r);
      if (c == b.counted.end()) return b.rules[r];
      auto it = counted_fsm.find(r);
      if (it == counted_fsm.end()) it = counted_fsm.emplace(r, counted_automaton(c->second)).first;
      return it->second;
    };
    // keep only rules reachable from the root; counted rules go last, so that their states are the top of the
    // state numbering (an item's state word below FlatGrammar::rep_first needs no decoding)
    std::vector<int> new_id(R, -1), order;
    order.push_back(root); new_id[root] = 0;
    for (size_t q = 0; q < order.size(); ++q)
      for (auto& es : fsm_of(order[q]).out)
        for (const Edge& e : es) if (e.kind == Edge::kRef && new_id[e.rule] < 0) { new_id[e.rule] = (int)order.size(); order.push_back(e.rule); }
    std::stable_partition(order.begin() + 1, order.end(), [&](int r) { return !b.counted.count(r); });
    for (size_t k = 0; k < order.size(); ++k) new_id[order[k]] = (int)k;
    bool any_counted = false;
    for (int r : order) any_counted = any_counted || b.counted.count(r);
    FlatGrammar g;
    g.n_rules = (int)order.size();
    g.root_rule = 0;
    g.root_nullable = root_nullable ? 1 : 0;
    g.max_expanded_repeat = b.max_expanded;
    std::map<ByteSet, int> class_id;
    std::vector<int> base(g.n_rules);
    for (int k = 0; k < g.n_rules; ++k) { base[k] = g.n_states; g.n_states += fsm_of(order[k]).size(); }
    g.n_base_states = g.n_states;
    g.cedge_begin.push_back(0); g.redge_begin.push_back(0);
    if (any_counted) { g.rule_rep_lo.assign(g.n_rules, 0); g.rule_rep_hi.assign(g.n_rules, 0); g.rep_depth = opt.repeat_depth; }
    for (int k = 0; k < g.n_rules; ++k) {
      const Fsm& f = fsm_of(order[k]);
      g.rule_names.push_back(b.names[order[k]]);
      g.rule_start.push_back(base[k] + f.start);
      g.rule_kind.push_back(f.has_tag_dispatch ? 1 : 0);
      auto c = b.counted.find(order[k]);
      if (c != b.counted.end()) {
        g.rule_rep_lo[k] = c->second.lo; g.rule_rep_hi[k] = c->second.hi;
        if (g.rep_first == 0x7FFFFFFF) g.rep_first = base[k];
      }
      for (int s = 0; s < f.size(); ++s) {
        g.state_rule.push_back(k);
        g.state_final.push_back(f.fin[s] ? 1 : 0);
        for (const Edge& e : f.out[s]) {
          if (e.kind == Edge::kBytes) {
            auto it = class_id.find(e.set);
            if (it == class_id.end()) {
              it = class_id.emplace(e.set, (int)class_id.size()).first;
              g.class_bits.insert(g.class_bits.end(), e.set.w.begin(), e.set.w.end());
            }
            g.cedge_class.push_back(it->second);
            g.cedge_target.push_back(base[k] + e.to);
            if (any_counted) g.cedge_iter.push_back(e.iter ? 1 : 0);
          } else if (e.kind == Edge::kRef) {
            g.redge_rule.push_back(new_id[e.rule]);
            g.redge_target.push_back(base[k] + e.to);
            if (any_counted) g.redge_iter.push_back(e.iter ? 1 : 0);
          }
        }
        g.cedge_begin.push_back((int)g.cedge_class.size());
        g.redge_begin.push_back((int)g.redge_rule.size());
      }
    }
    g.n_classes = (int)class_id.size();
    build_closure_lists(g);
    return g;
  }

  static void build_closure_lists(FlatGrammar& g) {
    int R = g.n_rules, S = g.n_states;
    // rules predicted transitively when rule r is predicted (r itself included)
    std::vector<std::vector<int>> closure(R);
    for (int r = 0; r < R; ++r) {
      std::vector<char> seen(R, 0);
      std::vector<int> stack{r};
      seen[r] = 1;
      while (!stack.empty()) {
        int u = stack.back(); stack.pop_back();
        closure[r].push_back(u);
        int s0 = g.rule_start[u];
        for (int e = g.redge_begin[s0]; e < g.redge_begin[s0 + 1]; ++e) if (!seen[g.redge_rule[e]]) { seen[g.redge_rule[e]] = 1; stack.push_back(g.redge_rule[e]); }
      }
    }
    g.scan_begin.assign(1, 0); g.wait_begin.assign(1, 0); g.gather_begin.assign(1, 0);
    g.scan_own_end.clear();
    g.scan_class.clear(); g.scan_target.clear(); g.wait_rule.clear(); g.wait_target.clear(); g.gather_state.clear();
    // what the device follows along an edge: the target state, or in the device view of a grammar with counted
    // repetitions the packed word (an edge copied from a predicted start state begins at count 0: no count flags)
    auto cword = [&](int e) { return g.cedge_word.empty() ? (uint32_t)g.cedge_target[e] : g.cedge_word[e]; };
    auto rword = [&](int e) { return g.redge_word.empty() ? (uint32_t)g.redge_target[e] : g.redge_word[e]; };
    std::vector<int> predicted;
    std::vector<char> mark(R, 0);
    for (int s = 0; s < S; ++s) {
      predicted.clear();
      for (int e = g.redge_begin[s]; e < g.redge_begin[s + 1]; ++e)
        for (int r : closure[g.redge_rule[e]]) if (!mark[r]) { mark[r] = 1; predicted.push_back(r); }
      std::sort(predicted.begin(), predicted.end());
      for (int r : predicted) mark[r] = 0;
      for (int e = g.cedge_begin[s]; e < g.cedge_begin[s + 1]; ++e) { g.scan_class.push_back(g.cedge_class[e]); g.scan_target.push_back(cword(e)); }
      g.scan_own_end.push_back((int)g.scan_class.size());
      for (int e = g.redge_begin[s]; e < g.redge_begin[s + 1]; ++e) { g.wait_rule.push_back(g.redge_rule[e]); g.wait_target.push_back(rword(e)); }
      if (g.cedge_begin[s + 1] > g.cedge_begin[s]) g.gather_state.push_back(s);
      for (int r : predicted) {
        int s0 = g.rule_start[r];
        for (int e = g.cedge_begin[s0]; e < g.cedge_begin[s0 + 1]; ++e) { g.scan_class.push_back(g.cedge_class[e]); g.scan_target.push_back((cword(e) & kTargetMask) | kSelfBit); }
        for (int e = g.redge_begin[s0]; e < g.redge_begin[s0 + 1]; ++e) { g.wait_rule.push_back(g.redge_rule[e]); g.wait_target.push_back((rword(e) & kTargetMask) | kSelfBit); }
        if (g.cedge_begin[s0 + 1] > g.cedge_begin[s0]) g.gather_state.push_back((int32_t)((uint32_t)s0 | kSelfBit));
      }
      g.scan_begin.push_back((int)g.scan_class.size());
      g.wait_begin.push_back((int)g.wait_rule.size());
      g.gather_begin.push_back((int)g.gather_state.size());
    }
    g.state_first.assign((size_t)S * 8, 0);
    for (int s = 0; s < S; ++s)
      for (int e = g.scan_begin[s]; e < g.scan_begin[s + 1]; ++e)
        for (int w = 0; w < 8; ++w) g.state_first[(size_t)s * 8 + w] |= g.class_bits[(size_t)g.scan_class[e] * 8 + w];
    g.rule_follow.assign((size_t)R * 8, 0);
    bool changed = true;
    while (changed) {
      changed = false;
      for (int s = 0; s < S; ++s)
        for (int e = g.redge_begin[s]; e < g.redge_begin[s + 1]; ++e) {
          const int r = g.redge_rule[e], t = g.redge_target[e];
          for (int w = 0; w < 8; ++w) {
            uint32_t add = g.state_first[(size_t)t * 8 + w];
            if (g.state_final[t]) add |= g.rule_follow[(size_t)g.state_rule[t] * 8 + w];
            uint32_t& dst = g.rule_follow[(size_t)r * 8 + w];
            if ((dst | add) != dst) { dst |= add; changed = true; }
          }
        }
    }
  }
};

// ------------------------------------------------------------------------------------------
// a small JSON reader (for schemas and TagDispatch specs)
// ------------------------------------------------------------------------------------------
struct Json {
  enum Type { kNull, kBool, kNumber, kString, kArray, kObject } type = kNull;
  bool boolean = false;
  std::string text;                                   // string value, or the number's source text
  std::vector<Json> items;
  std::vector<std::pair<std::string, Json>> members;  // declaration order kept
  const Json* get(const std::string& key) const {
    for (auto& m : members) if (m.first == key) return &m.second;
    return nullptr;
  }
};
class JsonReader {
 public:
  explicit JsonReader(const std::string& s) : s_(s) {}
  Json run() { Json v = value(0); ws(); if (i_ != s_.size()) err("trailing characters"); return v; }

 private:
  const std::string& s_;
  size_t i_ = 0;
  [[noreturn]] void err(const std::string& m) { fail(XG_ERR_PARSE, "JSON: " + m + " at offset " + std::to_string(i_)); }
  void ws() { while (i_ < s_.size() && (s_[i_] == ' ' || s_[i_] == '\t' || s_[i_] == '\n' || s_[i_] == '\r')) ++i_; }
  bool eat(char c) { ws(); if (i_ < s_.size() && s_[i_] == c) { ++i_; return true; } return false; }
  uint32_t hex4() {
    uint32_t v = 0;
    for (int k = 0; k < 4; ++k) {
      if (i_ >= s_.size() || !isxdigit((unsigned char)s_[i_])) err("bad \\u escape");
      char h = s_[i_++];
      v = v * 16 + (uint32_t)(isdigit((unsigned char)h) ? h - '0' : tolower(h) - 'a' + 10);
    }
    return v;
  }
  std::string string() {
    if (!eat('"')) err("expected a string");
    std::string out;
    while (true) {
      if (i_ >= s_.size()) err("unterminated string");
      unsigned char c = s_[i_++];
      if (c == '"') return out;
      if (c < 0x20) err("control character in string");
      if (c != '\\') { out += (char)c; continue; }
      if (i_ >= s_.size()) err("dangling backslash");
      char e = s_[i_++];
      switch (e) {
        case '"': case '\\': case '/': out += e; break;
        case 'b': out += '\b'; break; case 'f': out += '\f'; break; case 'n': out += '\n'; break;
        case 'r': out += '\r'; break; case 't': out += '\t'; break;
        case 'u': {
          uint32_t cp = hex4();
          if (cp >= 0xD800 && cp <= 0xDBFF && s_.compare(i_, 2, "\\u") == 0) { i_ += 2; uint32_t lo = hex4(); cp = 0x10000 + ((cp - 0xD800) << 10) + (lo - 0xDC00); }
          put_utf8(out, cp);
          break;
        }
        default: err("unknown escape");
      }
    }
  }
  Json value(int depth) {
    if (depth > 64) err("nesting too deep");
    ws();
    if (i_ >= s_.size()) err("unexpected end");
    Json v;
    char c = s_[i_];
    if (c == '{') {
      ++i_; v.type = Json::kObject;
      if (eat('}')) return v;
      do { std::string k = string(); if (!eat(':')) err("expected ':'"); v.members.emplace_back(k, value(depth + 1)); } while (eat(','));
      if (!eat('}')) err("expected '}'");
    } else if (c == '[') {
      ++i_; v.type = Json::kArray;
      if (eat(']')) return v;
      do v.items.push_back(value(depth + 1)); while (eat(','));
      if (!eat(']')) err("expected ']'");
    } else if (c == '"') { v.type = Json::kString; v.text = string(); }
    else if (s_.compare(i_, 4, "true") == 0) { v.type = Json::kBool; v.boolean = true; i_ += 4; }
    else if (s_.compare(i_, 5, "false") == 0) { v.type = Json::kBool; i_ += 5; }
    else if (s_.compare(i_, 4, "null") == 0) { i_ += 4; }
    else {
      size_t j = i_;
      while (j < s_.size() && (isdigit((unsigned char)s_[j]) || strchr("+-.eE", s_[j]))) ++j;
      if (j == i_) err("unexpected character");
      v.type = Json::kNumber; v.text = s_.substr(i_, j - i_); i_ = j;
    }
    return v;
  }
};

// JSON text of a string value as it must appear in generated output: short escapes for the
// usual controls, \u00XX for the rest, everything else verbatim
std::string json_string_text(const std::string& s) {
  std::string out = "\"";
  for (unsigned char c : s) {
    switch (c) {
      case '"': out += "\\\""; break; case '\\': out += "\\\\"; break;
      case '\n': out += "\\n"; break; case '\r': out += "\\r"; break; case '\t': out += "\\t"; break;
      case '\b': out += "\\b"; break; case '\f': out += "\\f"; break;
      default:
        if (c < 0x20) { char buf[8]; snprintf(buf, sizeof buf, "\\u%04x", c); out += buf; }
        else out += (char)c;
    }
  }
  return out + "\"";
}
// a grammar-text literal for exact bytes
std::string literal(const std::string& bytes) {
  std::string out = "\"";
  for (unsigned char c : bytes) {
    if (c == '"' || c == '\\') { out += '\\'; out += (char)c; }
    else if (c < 0x20 || c == 0x7F) { char buf[8]; snprintf(buf, sizeof buf, "\\x%02x", c); out += buf; }
    else out += (char)c;
  }
  return out + "\"";
}

// JSON schema subset -> grammar text.  Objects list all their properties, in order, separated by
// ", " with ": " after the key; strings, numbers, arrays as in JSON; bounds become repetitions
// (Section 3.6: minLength / maxLength / minItems / maxItems generate repetition structures).
class SchemaLowering {
 public:
  SchemaLowering(const Json* defs, std::string prefix) : defs_(defs), prefix_(std::move(prefix)) {}
  std::vector<std::string> rules;

  std::string lower(const Json& s) {
    if (s.type != Json::kObject) fail(XG_ERR_UNSUPPORTED, "schema: expected an object");
    if (const Json* ref = s.get("$ref")) {
      const std::string pre = "#/$defs/";
      if (ref->type != Json::kString || ref->text.compare(0, pre.size(), pre) != 0) fail(XG_ERR_UNSUPPORTED, "schema: only #/$defs/ references are supported");
      std::string name = ref->text.substr(pre.size());
      const Json* target = defs_ ? defs_->get(name) : nullptr;
      if (!target) fail(XG_ERR_PARSE, "schema: unknown reference " + ref->text);
      auto it = def_rule_.find(name);
      if (it != def_rule_.end()) return it->second;
      std::string rule = fresh("ref");
      def_rule_[name] = rule;
      std::string body = lower(*target);
      rules.push_back(rule + " ::= " + body);
      return rule;
    }
    if (const Json* en = s.get("enum")) {
      if (en->type != Json::kArray || en->items.empty()) fail(XG_ERR_UNSUPPORTED, "schema: enum must be a non-empty array");
      std::string out = "(";
      for (size_t k = 0; k < en->items.size(); ++k) {
        const Json& v = en->items[k];
        std::string text;
        if (v.type == Json::kString) text = json_string_text(v.text);
        else if (v.type == Json::kNumber) text = v.text;
        else if (v.type == Json::kBool) text = v.boolean ? "true" : "false";
        else if (v.type == Json::kNull) text = "null";
        else fail(XG_ERR_UNSUPPORTED, "schema: enum values must be scalars");
        out += (k ? " | " : " ") + literal(text);
      }
      return out + " )";
    }
    static const char* known[] = {"type", "properties", "required", "items", "minItems", "maxItems", "minLength", "maxLength", "$defs", "additionalProperties", "description", "title"};
    for (auto& m : s.members) {
      bool ok = false;
      for (const char* k : known) ok = ok || m.first == k;
      if (!ok) fail(XG_ERR_UNSUPPORTED, "schema: unsupported keyword " + m.first);
    }
    const Json* type = s.get("type");
    if (!type || type->type != Json::kString) fail(XG_ERR_UNSUPPORTED, "schema: missing type");
    const std::string& t = type->text;
    if (t == "object") return object(s);
    if (t == "array") return array(s);
    if (t == "string") {
      int lo = bound(s, "minLength", 0), hi = bound(s, "maxLength", -1);
      if (hi >= 0 && hi < lo) fail(XG_ERR_PARSE, "schema: maxLength < minLength");
      std::string key = "string_" + std::to_string(lo) + "_" + (hi < 0 ? std::string("inf") : std::to_string(hi));
      return shared(key, "\"\\\"\" " + char_rule() + repetition(lo, hi) + " \"\\\"\"");
    }
    if (t == "integer") return shared("integer", "\"-\"? ( \"0\" | [1-9] [0-9]* )");
    if (t == "number") return shared("number", "\"-\"? ( \"0\" | [1-9] [0-9]* ) ( \".\" [0-9]+ )? ( [eE] [+\\-]? [0-9]+ )?");
    if (t == "boolean") return shared("boolean", "\"true\" | \"false\"");
    if (t == "null") return shared("null", "\"null\"");
    fail(XG_ERR_UNSUPPORTED, "schema: unsupported type " + t);
  }

 private:
  const Json* defs_;
  std::string prefix_;
  std::map<std::string, std::string> def_rule_, shared_rule_;
  int counter_ = 0;
  std::string fresh(const std::string& hint) { return prefix_ + hint + "_" + std::to_string(++counter_); }
  std::string shared(const std::string& hint, const std::string& body) {
    auto it = shared_rule_.find(hint);
    if (it != shared_rule_.end()) return it->second;
    std::string rule = prefix_ + "json_" + hint;
    shared_rule_[hint] = rule;
    rules.push_back(rule + " ::= " + body);
    return rule;
  }
  std::string char_rule() { return shared("char", "[^\"\\\\\\x00-\\x1f] | \"\\\\\" ( [\"\\\\/bfnrt] | \"u\" [0-9a-fA-F]{4} )"); }
  static int bound(const Json& s, const char* key, int dflt) {
    const Json* v = s.get(key);
    if (!v) return dflt;
    if (v->type != Json::kNumber) fail(XG_ERR_PARSE, std::string("schema: ") + key + " must be a number");
    int n = atoi(v->text.c_str());
    if (n < 0 || n > 100000) fail(XG_ERR_UNSUPPORTED, std::string("schema: ") + key + " out of range");
    return n;
  }
  static std::string repetition(int lo, int hi) {
    if (hi < 0) return lo == 0 ? "*" : "{" + std::to_string(lo) + ",}";
    return "{" + std::to_string(lo) + "," + std::to_string(hi) + "}";
  }
  std::string object(const Json& s) {
    const Json* props = s.get("properties");
    const Json* req = s.get("required");
    if (const Json* ap = s.get("additionalProperties")) if (ap->type != Json::kBool || ap->boolean) fail(XG_ERR_UNSUPPORTED, "schema: additionalProperties must be false");
    if (props && props->type != Json::kObject) fail(XG_ERR_PARSE, "schema: properties must be an object");
    size_t n = props ? props->members.size() : 0;
    if (req) {
      if (req->type != Json::kArray || req->items.size() != n) fail(XG_ERR_UNSUPPORTED, "schema: every property must be required, in declared order");
      for (size_t k = 0; k < n; ++k) if (req->items[k].type != Json::kString || req->items[k].text != props->members[k].first) fail(XG_ERR_UNSUPPORTED, "schema: every property must be required, in declared order");
    }
    if (n == 0) return "\"{}\"";
    std::string body;
    for (size_t k = 0; k < n; ++k) {
      std::string lead = (k ? ", " : "{") + json_string_text(props->members[k].first) + ": ";
      body += literal(lead) + " " + lower(props->members[k].second) + " ";
    }
    body += "\"}\"";
    std::string rule = fresh("object");
    rules.push_back(rule + " ::= " + body);
    return rule;
  }
  std::string array(const Json& s) {
    const Json* items = s.get("items");
    if (!items) fail(XG_ERR_UNSUPPORTED, "schema: array without items");
    int lo = bound(s, "minItems", 0), hi = bound(s, "maxItems", -1);
    if (hi >= 0 && hi < lo) fail(XG_ERR_PARSE, "schema: maxItems < minItems");
    if (hi == 0) return "\"[]\"";
    std::string item = lower(*items);
    std::string more = "( \", \" " + item + " )" + repetition(std::max(lo - 1, 0), hi < 0 ? -1 : hi - 1);
    std::string rule = fresh("array");
    if (lo == 0) rules.push_back(rule + " ::= \"[\" ( " + item + " " + more + " )? \"]\"");
    else rules.push_back(rule + " ::= \"[\" " + item + " " + more + " \"]\"");
    return rule;
  }
};

}  // namespace

std::string json_schema_to_ebnf(const std::string& schema_json, const std::string& root_name, const std::string& prefix) {
  Json schema = JsonReader(schema_json).run();
  SchemaLowering low(schema.get("$defs"), prefix);
  std::string body = low.lower(schema);
  std::string out = root_name + " ::= " + body + "\n";
  for (auto& r : low.rules) out += r + "\n";
  return out;
}

std::string tag_dispatch_to_ebnf(const std::string& spec_json) {
  Json spec = JsonReader(spec_json).run();
  const Json* tags = spec.get("tags");
  if (!tags || tags->type != Json::kArray || tags->items.empty()) fail(XG_ERR_PARSE, "TagDispatch spec: \"tags\" must be a non-empty array");
  std::string rules, pairs;
  for (size_t ti = 0; ti < tags->items.size(); ++ti) {
    const Json& tag = tags->items[ti];
    const Json* text = tag.get("tag");
    const Json* tools = tag.get("tools");
    const Json* end = tag.get("end");
    if (!text || text->type != Json::kString || text->text.empty()) fail(XG_ERR_PARSE, "TagDispatch spec: missing tag string");
    const Json* free_text = tag.get("text");
    if (free_text && free_text->type == Json::kBool && free_text->boolean) {
      // a channel whose body is free text up to its end marker: a TagDispatch without tags that stops at the marker
      if (!end || end->type != Json::kString || end->text.empty()) fail(XG_ERR_PARSE, "TagDispatch spec: a text channel needs a non-empty \"end\"");
      std::string rule = "dispatch_" + std::to_string(ti);
      rules += rule + " ::= TagDispatch(stop_strs=(" + literal(end->text) + "))\n";
      pairs += (ti ? ", " : "") + std::string("(") + literal(text->text) + ", " + rule + ")";
      continue;
    }
    if (!tools || tools->type != Json::kArray || tools->items.empty()) fail(XG_ERR_PARSE, "TagDispatch spec: \"tools\" must be a non-empty array");
    std::string calls;
    for (size_t k = 0; k < tools->items.size(); ++k) {
      const Json* name = tools->items[k].get("name");
      const Json* schema = tools->items[k].get("schema");
      if (!name || name->type != Json::kString || !schema) fail(XG_ERR_PARSE, "TagDispatch spec: a tool needs \"name\" and \"schema\"");
      std::string prefix = "tool" + std::to_string(ti) + "_" + std::to_string(k) + "_";
      SchemaLowering low(schema->get("$defs"), prefix);
      std::string args = low.lower(*schema);
      for (auto& r : low.rules) rules += r + "\n";
      const Json* bare = tag.get("bare");
      if (bare && bare->type == Json::kBool && bare->boolean) rules += prefix + "call ::= " + args + "\n";      // the tag names the tool: arguments only
      else rules += prefix + "call ::= " + literal("{\"name\": " + json_string_text(name->text) + ", \"arguments\": ") + " " + args + " \"}\"\n";
      calls += (k ? " | " : "") + prefix + "call";
    }
    std::string rule = "dispatch_" + std::to_string(ti);
    rules += rule + " ::= ( " + calls + " ) " + literal(end && end->type == Json::kString ? end->text : "") + "\n";
    pairs += (ti ? ", " : "") + std::string("(") + literal(text->text) + ", " + rule + ")";
  }
  std::string stops;
  if (const Json* ss = spec.get("stop_strs")) {
    if (ss->type != Json::kArray) fail(XG_ERR_PARSE, "TagDispatch spec: stop_strs must be an array");
    for (size_t k = 0; k < ss->items.size(); ++k) stops += (k ? ", " : "") + literal(ss->items[k].text);
  }
  return "root ::= TagDispatch(" + pairs + ", stop_strs=(" + stops + "))\n" + rules;
}

FlatGrammar compile_frontend(int kind, const std::string& text, const std::string& root, const FrontendOptions& opt) {
  std::string ebnf;
  if (kind == kEbnf) ebnf = text;
  else if (kind == kJsonSchema) ebnf = json_schema_to_ebnf(text, "root", "");
  else if (kind == kTagDispatchJson) ebnf = tag_dispatch_to_ebnf(text);
  else fail(XG_ERR_INVALID_ARG, "unknown grammar kind");

  auto parsed = GrammarParser(Lexer(ebnf).run()).run();
  Compiler c;
  c.opt = opt;
  for (auto& r : parsed) {
    if (c.b.ids.count(r.first)) fail(XG_ERR_PARSE, "grammar text: rule defined twice: " + r.first);
    c.b.ids[r.first] = (int)c.b.names.size();
    c.b.names.push_back(r.first);
  }
  std::string root_name = (kind == kEbnf && !root.empty()) ? root : "root";
  c.root = c.b.lookup(root_name);
  c.b.max_states = opt.max_rule_states;
  if (opt.repeat_threshold > 0 && opt.repeat_depth <= 0) fail(XG_ERR_INVALID_ARG, "counted repetitions need the longest token's length");
  c.b.repeat_threshold = opt.repeat_threshold;
  for (auto& r : parsed) {
    Fsm f;
    auto p = c.b.frag(f, *r.second);
    f.start = p.first;
    f.fin[p.second] = 1;
    if (f.size() > opt.max_rule_states) fail(XG_ERR_CAPACITY, "rule " + r.first + " exceeds max_rule_states");
    c.b.rules.push_back(std::move(f));
  }
  for (auto& kv : c.b.pending) {              // the rules behind counted repetitions, in the order of their ids
    if (kv.first != c.n_rules()) fail(XG_ERR_INVALID_ARG, "internal: rule numbering");
    c.b.rules.push_back(std::move(kv.second));
  }
  c.b.pending.clear();
  c.remove_nullability();
  for (Fsm& f : c.b.rules) f = normalize(f, opt.max_rule_states);
  std::vector<char> stale = c.trim(), renormalized;           // stale: trimmed since it was last minimised
  c.inline_small_rules(renormalized);
  const std::vector<char> trimmed_again = c.trim();
  for (int r = 0; r < c.n_rules(); ++r)
    if (trimmed_again[r] || (stale[r] && !renormalized[r])) c.b.rules[r] = canonical_order(minimize(c.b.rules[r]));
  return c.flatten();
}

// ------------------------------------------------------------------------------------------
// Counted repetitions on the device (Section 3.6).  An item of X{lo,hi} is (state of X, origin, k).  How a token of
// at most L bytes behaves from it depends on k only through how far k + 1 is from the two bounds, and only up to L
// iterations away (every iteration consumes a byte), so the states are written out once per class
//   (dl, dr) = (min(max(lo - k - 1, 0), D), min(hi - k - 1, D)),   D = L + 1:
// the record is accepting iff X's state is and dl = 0, it has the iteration edges iff dr > 0, and its cache entry
// is exact for every count of the class.  The number of records depends on D, not on the bounds.
// ------------------------------------------------------------------------------------------
namespace {
struct CountClass { int dl, dr; };
CountClass count_class(int lo, int hi, int D, int k) {
  const int done = k + 1;
  return {std::min(std::max(lo - done, 0), D), std::min(hi - done, D)};
}
// the largest count of class (dl, dr), or -1 when no count in [0, hi) falls into it
int class_largest_count(int lo, int hi, int D, int dl, int dr) {
  int done_min = 1, done_max = hi;
  if (dl == D) done_max = std::min(done_max, lo - D);
  else if (dl == 0) done_min = std::max(done_min, lo);
  else { done_min = std::max(done_min, lo - dl); done_max = std::min(done_max, lo - dl); }
  if (dr == D) done_max = std::min(done_max, hi - D);
  else { done_min = std::max(done_min, hi - dr); done_max = std::min(done_max, hi - dr); }
  return done_min <= done_max ? done_max - 1 : -1;
}
}  // namespace

int32_t record_of(const FlatGrammar& r, int32_t q, int32_t k) {
  if (q < r.rep_first) return q;
  const int i = q - r.rep_first, D = r.rep_depth;
  const CountClass c = count_class(r.rep_lo[i], r.rep_hi[i], D, k);
  return r.rep_rec_base[i] + c.dl * (D + 1) + c.dr;
}

FlatGrammar expand_counted_rules(const FlatGrammar& g) {
  if (g.rule_rep_lo.empty()) return g;
  const int D = g.rep_depth, per = (D + 1) * (D + 1);
  const int n_rep = g.n_base_states - g.rep_first;
  FlatGrammar r;
  r.n_rules = g.n_rules; r.n_classes = g.n_classes; r.root_rule = g.root_rule; r.root_nullable = g.root_nullable;
  r.rule_names = g.rule_names; r.rule_kind = g.rule_kind; r.class_bits = g.class_bits;
  r.rule_rep_lo = g.rule_rep_lo; r.rule_rep_hi = g.rule_rep_hi;
  r.rep_first = g.rep_first; r.rep_depth = D; r.n_base_states = g.n_base_states; r.max_expanded_repeat = g.max_expanded_repeat;
  r.rep_shift = 1;
  while ((1ll << r.rep_shift) < g.n_base_states) ++r.rep_shift;
  int hi_max = 0;
  for (int x : g.rule_rep_hi) hi_max = std::max(hi_max, x);
  if (r.rep_shift > 28 || (long long)hi_max >= (1ll << (32 - r.rep_shift))) fail(XG_ERR_CAPACITY, "a repetition bound does not fit the item's count field");
  const long long n_states = (long long)g.rep_first + (long long)n_rep * per;
  if (n_states > (long long)kTargetMask) fail(XG_ERR_CAPACITY, "too many state records");
  r.n_states = (int)n_states;
  r.rep_rec_base.resize(n_rep); r.rep_lo.resize(n_rep); r.rep_hi.resize(n_rep);
  for (int i = 0; i < n_rep; ++i) {
    const int rule = g.state_rule[g.rep_first + i];
    r.rep_rec_base[i] = g.rep_first + i * per; r.rep_lo[i] = g.rule_rep_lo[rule]; r.rep_hi[i] = g.rule_rep_hi[rule];
  }
  r.cedge_begin.push_back(0); r.redge_begin.push_back(0);
  r.rec_word.reserve(r.n_states);
  for (int s = 0; s < g.rep_first; ++s) {           // ordinary states: as they are
    r.state_rule.push_back(g.state_rule[s]); r.state_final.push_back(g.state_final[s]); r.rec_word.push_back((uint32_t)s);
    for (int e = g.cedge_begin[s]; e < g.cedge_begin[s + 1]; ++e) { r.cedge_class.push_back(g.cedge_class[e]); r.cedge_target.push_back(record_of(r, g.cedge_target[e], 0)); r.cedge_word.push_back((uint32_t)g.cedge_target[e]); }
    for (int e = g.redge_begin[s]; e < g.redge_begin[s + 1]; ++e) { r.redge_rule.push_back(g.redge_rule[e]); r.redge_target.push_back(record_of(r, g.redge_target[e], 0)); r.redge_word.push_back((uint32_t)g.redge_target[e]); }
    r.cedge_begin.push_back((int)r.cedge_class.size()); r.redge_begin.push_back((int)r.redge_rule.size());
  }
  for (int i = 0; i < n_rep; ++i) {
    const int q = g.rep_first + i, lo = r.rep_lo[i], hi = r.rep_hi[i];
    for (int dl = 0; dl <= D; ++dl)
      for (int dr = 0; dr <= D; ++dr) {
        const int k = class_largest_count(lo, hi, D, dl, dr);
        r.state_rule.push_back(g.state_rule[q]);
        r.state_final.push_back(k >= 0 && g.state_final[q] && dl == 0 ? 1 : 0);
        r.rec_word.push_back((uint32_t)q | (k >= 0 ? (uint32_t)k << r.rep_shift : 0u));
        if (k >= 0) {
          for (int e = g.cedge_begin[q]; e < g.cedge_begin[q + 1]; ++e) {
            const bool iter = g.cedge_iter[e] != 0;
            if (iter && dr == 0) continue;
            r.cedge_class.push_back(g.cedge_class[e]);
            r.cedge_target.push_back(record_of(r, g.cedge_target[e], iter ? k + 1 : k));
            r.cedge_word.push_back((uint32_t)g.cedge_target[e] | kRelBit | (iter ? kIterBit : 0u));
          }
          for (int e = g.redge_begin[q]; e < g.redge_begin[q + 1]; ++e) {
            const bool iter = g.redge_iter[e] != 0;
            if (iter && dr == 0) continue;
            r.redge_rule.push_back(g.redge_rule[e]);
            r.redge_target.push_back(record_of(r, g.redge_target[e], iter ? k + 1 : k));
            r.redge_word.push_back((uint32_t)g.redge_target[e] | kRelBit | (iter ? kIterBit : 0u));
          }
        }
        r.cedge_begin.push_back((int)r.cedge_class.size()); r.redge_begin.push_back((int)r.redge_rule.size());
      }
  }
  for (int rule = 0; rule < g.n_rules; ++rule) r.rule_start.push_back(record_of(r, g.rule_start[rule], 0));
  Compiler::build_closure_lists(r);
  // follow sets from the plain automata (every edge enabled, acceptance as in X): a superset for every count
  r.rule_follow = g.rule_follow;
  return r;
}


// Repetition state compression (Section 3.6), as an equivalence on automaton states.  A cache
// entry only records how tokens of at most `depth` bytes behave from its state, so two states of
// one rule whose automata agree when unrolled `depth` edges deep (every edge consumes at least
// one byte: no rule derives the empty string) have the same entry.  Inside a bounded repetition
// R{l,r} almost all copies of R are alike in this sense -- only the copies within `depth` of the
// bounds differ -- so the number of entries to build stays bounded however large r is, while the
// explicit states keep the exact count k of (R{l,r}, k) for the run-time check.
//   level 0:   same rule, same acceptance;
//   level d+1: level 0, and the same edges (byte class or referenced rule) into level-d classes.
// Returns, per state, the smallest state of its class after `depth` rounds of refinement (a
// partition at least as fine as level `depth`, at most as fine as full bisimulation).
std::vector<int32_t> bounded_equivalence(const FlatGrammar& g, int depth) {
  const int S = g.n_states;
  // predecessors (CSR): whose signature goes stale when a state changes class
  std::vector<int> pred_begin(S + 1, 0), pred;
  for (int t : g.cedge_target) ++pred_begin[t + 1];
  for (int t : g.redge_target) ++pred_begin[t + 1];
  for (int s = 0; s < S; ++s) pred_begin[s + 1] += pred_begin[s];
  pred.resize(pred_begin[S]);
  {
    std::vector<int> at(pred_begin.begin(), pred_begin.end() - 1);
    for (int s = 0; s < S; ++s) {
      for (int e = g.cedge_begin[s]; e < g.cedge_begin[s + 1]; ++e) pred[at[g.cedge_target[e]]++] = s;
      for (int e = g.redge_begin[s]; e < g.redge_begin[s + 1]; ++e) pred[at[g.redge_target[e]]++] = s;
    }
  }
  // level 0
  std::vector<int> block(S), count;
  {
    SignatureTable table;
    std::vector<uint32_t> sig(3);
    for (int s = 0; s < S; ++s) {
      sig[0] = (uint32_t)g.state_rule[s]; sig[1] = g.state_final[s];
      sig[2] = s >= g.rep_first ? (uint32_t)s + 1 : 0u;        // the records of a counted rule are classes already
      block[s] = table.intern(sig);
      if (block[s] == (int)count.size()) count.push_back(0);
      ++count[block[s]];
    }
  }
  // One round per level.  A state's signature (its edges with targets replaced by their classes)
  // is recomputed only after one of its targets moved to a new class.  All members of a class
  // carry the same signature once a round is over, so a round only has to place the recomputed
  // states: those that still match their class's standing signature stay, every other group
  // becomes a new class (when the whole class was recomputed, its largest group keeps the id).
  // A round costs in proportion to what changed, not to S.
  SignatureTable table;
  std::vector<int> sig_id(S, -1), standing(count.size(), -1), work(S);
  std::vector<char> queued(S, 1);
  for (int s = 0; s < S; ++s) work[s] = s;
  std::vector<uint32_t> sig;
  std::vector<std::pair<uint32_t, uint32_t>> edges;
  std::vector<int> moved;
  for (int level = 0; level < depth && !work.empty(); ++level) {
    for (int s : work) {
      sig.clear();
      edges.clear();
      for (int e = g.cedge_begin[s]; e < g.cedge_begin[s + 1]; ++e) edges.emplace_back((uint32_t)g.cedge_class[e], (uint32_t)block[g.cedge_target[e]]);
      std::sort(edges.begin(), edges.end());
      sig.push_back((uint32_t)edges.size());
      for (auto& p : edges) { sig.push_back(p.first); sig.push_back(p.second); }
      edges.clear();
      for (int e = g.redge_begin[s]; e < g.redge_begin[s + 1]; ++e) edges.emplace_back((uint32_t)g.redge_rule[e], (uint32_t)block[g.redge_target[e]]);
      std::sort(edges.begin(), edges.end());
      for (auto& p : edges) { sig.push_back(p.first); sig.push_back(p.second); }
      sig_id[s] = table.intern(sig);
      queued[s] = 0;
    }
    std::sort(work.begin(), work.end(), [&](int x, int y) {
      if (block[x] != block[y]) return block[x] < block[y];
      return sig_id[x] != sig_id[y] ? sig_id[x] < sig_id[y] : x < y;
    });
    moved.clear();
    for (size_t lo = 0; lo < work.size();) {
      const int b = block[work[lo]];
      size_t hi = lo;
      while (hi < work.size() && block[work[hi]] == b) ++hi;
      int keep = standing[b];
      if ((int)(hi - lo) == count[b]) {               // nobody holds the standing signature any more: the largest group stays
        size_t best = 0;
        for (size_t i = lo; i < hi;) {
          size_t j = i;
          while (j < hi && sig_id[work[j]] == sig_id[work[i]]) ++j;
          if (j - i > best) { best = j - i; keep = sig_id[work[i]]; }
          i = j;
        }
        standing[b] = keep;
      }
      for (size_t i = lo; i < hi;) {
        size_t j = i;
        while (j < hi && sig_id[work[j]] == sig_id[work[i]]) ++j;
        if (sig_id[work[i]] != keep) {
          const int id = (int)count.size();
          count.push_back((int)(j - i));
          standing.push_back(sig_id[work[i]]);
          count[b] -= (int)(j - i);
          for (size_t k = i; k < j; ++k) { block[work[k]] = id; moved.push_back(work[k]); }
        }
        i = j;
      }
      lo = hi;
    }
    work.clear();
    for (int s : moved)
      for (int q = pred_begin[s]; q < pred_begin[s + 1]; ++q) if (!queued[pred[q]]) { queued[pred[q]] = 1; work.push_back(pred[q]); }
  }
  std::vector<int32_t> first(count.size(), -1), rep(S);
  for (int s = 0; s < S; ++s) { if (first[block[s]] < 0) first[block[s]] = s; rep[s] = first[block[s]]; }
  return rep;
}

}  // namespace xg
