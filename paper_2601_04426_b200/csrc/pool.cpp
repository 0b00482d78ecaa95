#include "pool.h"

#include <algorithm>
#include <memory>
#include <functional>
#include <iterator>

namespace xg {

// tags of Algorithm 1 (any distinct constants) and the placeholder of Algorithm 2
static const uint64_t kNodeTag = 0x4E4F44455F544147ull, kRangeTag = 0x52414E47455F5447ull, kRefTag = 0x5245465F5F544147ull,
                      kPlaceholder = 0x58585F484F4C4445ull, kSccRefTag = 0x5343435F5F524546ull, kRuleTag = 0x52554C455F544147ull;

uint64_t hash_fold(uint64_t h, uint64_t x) {
  uint64_t z = (h ^ x) + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

DeviceArena::~DeviceArena() {
  for (auto& s : slabs_) if (s.base) cudaFree(s.base);
}

void* DeviceArena::alloc(size_t bytes) {
  bytes = (std::max<size_t>(bytes, 1) + 255) & ~size_t(255);
  int slab = -1;
  size_t offset = 0;
  for (int i = 0; i < (int)slabs_.size() && slab < 0; ++i) {
    if (!slabs_[i].base || slabs_[i].bytes - slabs_[i].used < bytes) continue;
    for (auto& blk : slabs_[i].free_blocks)
      if (blk.second >= bytes) { slab = i; offset = blk.first; break; }
  }
  if (slab < 0) {
    const size_t want = std::max(bytes, std::min<size_t>(size_t(256) << 20, std::max<size_t>(size_t(1) << 20, reserved_)));
    void* base = nullptr;
    size_t got = want;
    if (cudaMalloc(&base, got) != cudaSuccess) {
      cudaGetLastError();
      got = bytes;
      if (got == want || cudaMalloc(&base, got) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    }
    for (slab = 0; slab < (int)slabs_.size() && slabs_[slab].base; ++slab) {}
    if (slab == (int)slabs_.size()) slabs_.emplace_back();
    Slab& s = slabs_[slab];
    s.base = (char*)base; s.bytes = got; s.used = 0;
    s.free_blocks.clear();
    s.free_blocks[0] = got;
    reserved_ += got;
    offset = 0;
  }
  Slab& s = slabs_[slab];
  const size_t len = s.free_blocks[offset];
  s.free_blocks.erase(offset);
  if (len > bytes) s.free_blocks[offset + bytes] = len - bytes;
  s.used += bytes;
  void* p = s.base + offset;
  live_[p] = std::make_pair(slab, bytes);
  return p;
}

bool DeviceArena::reserve(size_t bytes) {
  while (bytes > 0) {
    const size_t want = std::min<size_t>(bytes, size_t(1) << 30);
    void* base = nullptr;
    if (cudaMalloc(&base, want) != cudaSuccess) { cudaGetLastError(); return false; }
    int slab = 0;
    for (; slab < (int)slabs_.size() && slabs_[slab].base; ++slab) {}
    if (slab == (int)slabs_.size()) slabs_.emplace_back();
    Slab& s = slabs_[slab];
    s.base = (char*)base; s.bytes = want; s.used = 0; s.keep = true;
    s.free_blocks.clear();
    s.free_blocks[0] = want;
    reserved_ += want;
    bytes -= want;
  }
  return true;
}

void DeviceArena::free(void* p) {
  auto it = live_.find(p);
  if (it == live_.end()) return;
  const int slab = it->second.first;
  size_t bytes = it->second.second;
  live_.erase(it);
  Slab& s = slabs_[slab];
  s.used -= bytes;
  if (s.used == 0 && !s.keep) {          // nothing left in it: back to the driver
    cudaFree(s.base);
    reserved_ -= s.bytes;
    s = Slab();
    return;
  }
  size_t offset = (size_t)((char*)p - s.base);
  auto next = s.free_blocks.lower_bound(offset);
  if (next != s.free_blocks.end() && offset + bytes == next->first) { bytes += next->second; next = s.free_blocks.erase(next); }
  if (next != s.free_blocks.begin()) {
    auto prev = std::prev(next);
    if (prev->first + prev->second == offset) { prev->second += bytes; return; }
  }
  s.free_blocks[offset] = bytes;
}

CachePool::~CachePool() {
  for (auto& s : scratch_) cudaFree(s.first);
  for (auto& s : pinned_) if (s.first) cudaFreeHost(s.first);
  cudaFree(jit_.d_used);
  if (jit_host && jit_host_free) jit_host_free(jit_host);
  for (cudaEvent_t e : timing_) if (e) cudaEventDestroy(e);
}

cudaEvent_t* CachePool::timing_events() {
  if (!timing_[0]) {
    if (cudaEventCreate(&timing_[0]) != cudaSuccess) { timing_[0] = nullptr; return nullptr; }
    if (cudaEventCreate(&timing_[1]) != cudaSuccess) { cudaEventDestroy(timing_[0]); timing_[0] = timing_[1] = nullptr; return nullptr; }
  }
  return timing_;
}

const CachePool::JitArena* CachePool::jit_arena(long long min_words, bool renew, long long first_words) {
  if (jit_.base && !renew && jit_.cap_words >= min_words) return &jit_;
  // the old chunk stays in the pool for the entries already in it; new builds go to the new one
  long long words = std::max<long long>(min_words, jit_.base ? std::min<long long>(2 * jit_.cap_words, (64LL << 20)) : (first_words > 0 ? first_words : (8LL << 20)));
  JitArena a;
  a.base = (uint32_t*)allocate_device((size_t)words * 4, &a.chunk);
  if (!a.base) return nullptr;
  if (cudaMalloc(&a.d_used, sizeof(unsigned long long)) != cudaSuccess || cudaMemset(a.d_used, 0, sizeof(unsigned long long)) != cudaSuccess) {
    cudaFree(a.d_used);
    return nullptr;                      // the chunk stays registered and idle: the limit's eviction returns it
  }
  a.cap_words = words;
  cudaFree(jit_.d_used);
  jit_ = a;
  return &jit_;
}

void* CachePool::scratch(int slot, size_t bytes) {
  if ((int)scratch_.size() <= slot) scratch_.resize(slot + 1, {nullptr, 0});
  auto& s = scratch_[slot];
  if (s.second < bytes) {
    cudaFree(s.first);
    s = {nullptr, 0};
    size_t want = bytes + bytes / 4;
    if (cudaMalloc(&s.first, want) != cudaSuccess) { s.first = nullptr; return nullptr; }
    s.second = want;
  }
  return s.first;
}

void* CachePool::pinned(int slot, size_t bytes) {
  if ((int)pinned_.size() <= slot) pinned_.resize(slot + 1, {nullptr, 0});
  auto& s = pinned_[slot];
  if (s.second < bytes) {
    if (s.first) cudaFreeHost(s.first);
    s = {nullptr, 0};
    size_t want = bytes + bytes / 2;
    if (cudaHostAlloc(&s.first, want, cudaHostAllocDefault) != cudaSuccess) { s.first = nullptr; return nullptr; }
    s.second = want;
  }
  return s.first;
}

void* CachePool::allocate_device(size_t bytes, int* chunk_id) {
  void* p = arena_.alloc(bytes);
  if (!p) return nullptr;
  Chunk c;
  c.ptr = p; c.bytes = bytes; c.last_use = ++clock_;
  chunks_.push_back(c);
  bytes_ += (long long)bytes;
  *chunk_id = (int)chunks_.size() - 1;
  return p;
}

void CachePool::retain(const std::vector<int>& chunk_ids) {
  for (int c : chunk_ids) { ++chunks_[c].refs; chunks_[c].last_use = ++clock_; }
}

void CachePool::release(const std::vector<int>& chunk_ids) {
  std::lock_guard<std::mutex> lock(mu);
  release_held(chunk_ids);
}

void CachePool::release_held(const std::vector<int>& chunk_ids) {
  for (int c : chunk_ids) --chunks_[c].refs;
  enforce_limit();
}

void CachePool::enforce_limit() {
  if (limit_ <= 0) return;
  while (bytes_ > limit_) {
    int victim = -1;
    for (int c = 0; c < (int)chunks_.size(); ++c)
      if (chunks_[c].ptr && chunks_[c].refs == 0 && (victim < 0 || chunks_[c].last_use < chunks_[victim].last_use)) victim = c;
    if (victim < 0) return;               // everything left is in use
    Chunk& ch = chunks_[victim];
    for (int r : ch.rules) {              // the rules of this chunk leave the pool (a later compile rebuilds them)
      PoolRule& pr = rules_[r];
      if (!pr.built) continue;
      auto& bucket = by_hash_[pr.hash];
      bucket.erase(std::remove(bucket.begin(), bucket.end(), r), bucket.end());
      pr.built = false;
      pr.serial.clear(); pr.entries.clear(); pr.counts.clear(); pr.chunks.clear(); pr.have.clear();
    }
    if (victim == jit_.chunk) { cudaFree(jit_.d_used); jit_ = JitArena(); }
    cudaDeviceSynchronize();              // nothing may still be reading the chunk
    arena_.free(ch.ptr);
    bytes_ -= (long long)ch.bytes;
    ++evicted_chunks_; evicted_bytes_ += (long long)ch.bytes;
    ch.ptr = nullptr; ch.bytes = 0; ch.rules.clear();
  }
}

CachePool::Stats CachePool::stats() const {
  Stats s;
  s.bytes = bytes_; s.reserved = (long long)arena_.reserved(); s.evicted_chunks = evicted_chunks_; s.evicted_bytes = evicted_bytes_;
  for (auto& r : rules_) s.live_rules += r.built ? 1 : 0;
  for (auto& c : chunks_) s.chunks += c.ptr ? 1 : 0;
  return s;
}

int CachePool::find_or_add(uint64_t hash, std::vector<uint64_t>&& serial) {
  auto& bucket = by_hash_[hash];
  for (int id : bucket) if (rules_[id].serial == serial) return id;     // equal hash is not trusted on its own
  PoolRule r;
  r.hash = hash;
  r.serial = std::move(serial);
  rules_.push_back(std::move(r));
  bucket.push_back((int)rules_.size() - 1);
  return (int)rules_.size() - 1;
}

namespace {

struct OutEdge {
  bool is_ref;
  int lo, hi;       // byte range (a class edge is split into its maximal ranges)
  int rule;         // referenced rule
  int target;       // state offset inside the rule
};

struct RuleShape {
  int first = 0, n = 0;                       // states [first, first + n)
  std::vector<std::vector<OutEdge>> out;      // by state offset
  std::vector<char> fin;
  int start = 0;
};

RuleShape shape_of(const FlatGrammar& g, int r, int first, int n) {
  RuleShape sh;
  sh.first = first; sh.n = n; sh.start = g.rule_start[r] - first;
  sh.out.resize(n); sh.fin.resize(n);
  for (int k = 0; k < n; ++k) {
    const int s = first + k;
    sh.fin[k] = g.state_final[s];
    for (int e = g.cedge_begin[s]; e < g.cedge_begin[s + 1]; ++e) {
      const uint32_t* bits = &g.class_bits[(size_t)g.cedge_class[e] * 8];
      int b = 0;
      while (b < 256) {
        if (!((bits[b >> 5] >> (b & 31)) & 1u)) { ++b; continue; }
        int lo = b;
        while (b < 256 && ((bits[b >> 5] >> (b & 31)) & 1u)) ++b;
        sh.out[k].push_back({false, lo, b - 1, -1, g.cedge_target[e] - first});
      }
    }
    for (int e = g.redge_begin[s]; e < g.redge_begin[s + 1]; ++e) sh.out[k].push_back({true, 0, 0, g.redge_rule[e], g.redge_target[e] - first});
  }
  return sh;
}

// A key of a rule's automaton that does not depend on any numbering (of its states, of its edges or of the rules
// it refers to): sizes and a commutative sum over its byte ranges.  It orders references whose hashes are still
// equal -- the members of a cycle all carry the placeholder while the cycle is being hashed -- so that the same
// structure gets the same canonical order in every grammar, whatever indices its rules have there.
uint64_t shape_key(const RuleShape& sh) {
  uint64_t ranges = 0, refs = 0, finals = 0;
  for (int k = 0; k < sh.n; ++k) {
    finals += sh.fin[k] ? 1 : 0;
    for (const OutEdge& e : sh.out[k]) {
      if (e.is_ref) ++refs;
      else ranges += hash_fold(kRangeTag, ((uint64_t)e.lo << 8) | (uint64_t)e.hi);
    }
  }
  return hash_fold(hash_fold(hash_fold(hash_fold(0, (uint64_t)sh.n), finals), refs), ranges);
}

// The canonical order of a rule's states (Section 3.3: two automata of the same structure must be numbered alike
// before they can be hashed): out-edges sorted -- byte ranges by their bounds, references by the hash of the rule
// they name, then by that rule's shape key --, then a breadth-first search from the start state; a state's
// canonical id is its place in the order of discovery.  Returns canonical index -> state offset.
std::vector<int> canonical_states(RuleShape& sh, const std::vector<uint64_t>& ref_hash, const std::vector<uint64_t>& ref_key) {
  for (auto& es : sh.out)
    std::stable_sort(es.begin(), es.end(), [&](const OutEdge& a, const OutEdge& b) {
      if (a.is_ref != b.is_ref) return !a.is_ref;
      if (!a.is_ref) return a.lo != b.lo ? a.lo < b.lo : a.hi < b.hi;
      if (ref_hash[a.rule] != ref_hash[b.rule]) return ref_hash[a.rule] < ref_hash[b.rule];
      if (ref_key[a.rule] != ref_key[b.rule]) return ref_key[a.rule] < ref_key[b.rule];
      return a.rule < b.rule;
    });
  std::vector<int> order{sh.start}, id(sh.n, -1);
  id[sh.start] = 0;
  for (size_t q = 0; q < order.size(); ++q)
    for (const OutEdge& e : sh.out[order[q]]) if (id[e.target] < 0) { id[e.target] = (int)order.size(); order.push_back(e.target); }
  return order;
}

// The hash of a rule: its automaton written out in canonical order as a flat sequence of words -- per state a
// marker with the accepting flag, per edge its kind, its label (a byte range, or the hash of the referenced rule) and
// the canonical id of its target -- folded in one pass.  (The pool's exact identity check serialises the same way,
// with pool ids in place of hashes.)
uint64_t hash_rule(const RuleShape& sh, const std::vector<int>& order, const std::vector<uint64_t>& ref_hash) {
  std::vector<int> id(sh.n, -1);
  for (size_t k = 0; k < order.size(); ++k) id[order[k]] = (int)k;
  std::vector<uint64_t> words;
  for (int s : order) {
    words.push_back(kNodeTag);
    words.push_back(sh.fin[s] ? 1 : 0);
    for (const OutEdge& e : sh.out[s]) {
      words.push_back(e.is_ref ? kRefTag : kRangeTag);
      words.push_back(e.is_ref ? ref_hash[e.rule] : (((uint64_t)e.lo << 8) | (uint64_t)e.hi));
      words.push_back((uint64_t)id[e.target]);
    }
  }
  uint64_t h = 0;
  for (uint64_t w : words) h = hash_fold(h, w);
  return h;
}

struct Analysis {
  std::vector<RuleShape> shapes;
  std::vector<std::vector<int>> adj, comps;     // comps: strongly connected components, callees first
  std::vector<int> comp;
  RuleInterning out;
  bool cyclic(const std::vector<int>& members) const {
    return members.size() > 1 || std::binary_search(adj[members[0]].begin(), adj[members[0]].end(), members[0]);
  }
};

Analysis analyse(const FlatGrammar& g) {
  const int R = g.n_rules;
  Analysis a;
  RuleInterning& out = a.out;
  out.pool_id.assign(R, -1);
  out.canon.resize(R);
  out.hash.assign(R, 0);
  std::vector<int> first(R + 1, g.n_states);
  for (int s = g.n_states - 1; s >= 0; --s) first[g.state_rule[s]] = s;
  a.shapes.resize(R);
  for (int r = 0; r < R; ++r) a.shapes[r] = shape_of(g, r, first[r], first[r + 1] - first[r]);
  a.adj.resize(R);
  for (int r = 0; r < R; ++r) {
    for (auto& es : a.shapes[r].out) for (const OutEdge& e : es) if (e.is_ref) a.adj[r].push_back(e.rule);
    std::sort(a.adj[r].begin(), a.adj[r].end());
    a.adj[r].erase(std::unique(a.adj[r].begin(), a.adj[r].end()), a.adj[r].end());
  }
  // strongly connected components (Tarjan); components come out callees first
  std::vector<int> index(R, -1), low(R, 0), stack;
  a.comp.assign(R, -1);
  std::vector<char> on_stack(R, 0);
  int counter = 0;
  std::function<void(int)> dfs = [&](int u) {
    index[u] = low[u] = counter++;
    stack.push_back(u); on_stack[u] = 1;
    for (int w : a.adj[u]) {
      if (index[w] < 0) { dfs(w); low[u] = std::min(low[u], low[w]); }
      else if (on_stack[w]) low[u] = std::min(low[u], index[w]);
    }
    if (low[u] == index[u]) {
      a.comps.emplace_back();
      while (true) { int w = stack.back(); stack.pop_back(); on_stack[w] = 0; a.comp[w] = (int)a.comps.size() - 1; a.comps.back().push_back(w); if (w == u) break; }
    }
  };
  for (int r = 0; r < R; ++r) if (index[r] < 0) dfs(r);

  std::vector<uint64_t> ref_hash(R, kPlaceholder);     // unresolved references hash as the placeholder
  std::vector<uint64_t> ref_key(R);
  for (int r = 0; r < R; ++r) ref_key[r] = shape_key(a.shapes[r]);
  for (auto& members : a.comps) {
    if (!a.cyclic(members)) {
      const int r = members[0];
      out.canon[r] = canonical_states(a.shapes[r], ref_hash, ref_key);
      out.hash[r] = hash_rule(a.shapes[r], out.canon[r], ref_hash);
      ref_hash[r] = out.hash[r];
      continue;
    }
    // Local hashes with the placeholder on in-cycle references, then the refinement of
    // Algorithm 2: fold the local hashes starting from each member.  For a simple cycle the
    // members are visited in cycle order (the rotation of Algorithm 2); for a denser component,
    // in breadth-first order of the reference edges.
    std::vector<uint64_t> local(R, 0);
    for (int r : members) {
      out.canon[r] = canonical_states(a.shapes[r], ref_hash, ref_key);
      local[r] = hash_rule(a.shapes[r], out.canon[r], ref_hash);
    }
    for (int r : members) {
      std::vector<int> seq{r};
      std::vector<char> seen(R, 0);
      seen[r] = 1;
      for (size_t q = 0; q < seq.size(); ++q) {
        const RuleShape& sh = a.shapes[seq[q]];
        for (int s : out.canon[seq[q]])
          for (const OutEdge& e : sh.out[s]) if (e.is_ref && a.comp[e.rule] == a.comp[r] && !seen[e.rule]) { seen[e.rule] = 1; seq.push_back(e.rule); }
      }
      uint64_t h = 0;
      for (int m : seq) h = hash_fold(h, local[m]);
      out.hash[r] = h;
    }
    for (int r : members) ref_hash[r] = out.hash[r];
    // the hashes of in-cycle references changed the sort keys: fix the canonical orders again
    for (int r : members) out.canon[r] = canonical_states(a.shapes[r], ref_hash, ref_key);
  }
  return a;
}

}  // namespace

RuleInterning structural_hashes(const FlatGrammar& g) { return analyse(g).out; }

// the part of interning that needs no pool: shapes, canonical state orders, hashes
std::shared_ptr<const void> prepare_interning(const FlatGrammar& g) {
  return std::shared_ptr<const void>(new Analysis(analyse(g)), [](const void* p) { delete static_cast<const Analysis*>(p); });
}

RuleInterning CachePool::intern(const FlatGrammar& g, const std::shared_ptr<const void>& prepared) {
  Analysis a = prepared ? *static_cast<const Analysis*>(prepared.get()) : analyse(g);
  RuleInterning& out = a.out;
  const int R = g.n_rules;
  // exact identities: serialise each rule with its callees named by pool id; members of a
  // cycle are serialised jointly, named by discovery order from the rule being keyed
  for (auto& members : a.comps) {
    const bool cyclic = a.cyclic(members);
    for (int r : members) {
      std::vector<int> seq{r};
      std::vector<int> local_id(R, -1);
      local_id[r] = 0;
      std::vector<uint64_t> serial;
      for (size_t q = 0; q < seq.size(); ++q) {
        const int m = seq[q];
        const RuleShape& sh = a.shapes[m];
        std::vector<int> id(sh.n, -1);
        for (size_t k = 0; k < out.canon[m].size(); ++k) id[out.canon[m][k]] = (int)k;
        serial.push_back(kRuleTag);
        serial.push_back((uint64_t)out.canon[m].size());
        for (int s : out.canon[m]) {
          serial.push_back(kNodeTag); serial.push_back(sh.fin[s] ? 1 : 0);
          for (const OutEdge& e : sh.out[s]) {
            if (!e.is_ref) { serial.push_back(kRangeTag); serial.push_back(((uint64_t)e.lo << 8) | (uint64_t)e.hi); serial.push_back((uint64_t)id[e.target]); }
            else if (cyclic && a.comp[e.rule] == a.comp[r]) {
              if (local_id[e.rule] < 0) { local_id[e.rule] = (int)seq.size(); seq.push_back(e.rule); }
              serial.push_back(kSccRefTag); serial.push_back((uint64_t)local_id[e.rule]); serial.push_back((uint64_t)id[e.target]);
            } else { serial.push_back(kRefTag); serial.push_back((uint64_t)out.pool_id[e.rule]); serial.push_back((uint64_t)id[e.target]); }
          }
        }
      }
      // pool ids of cycle members are only read by rules outside the cycle, so they can be
      // assigned one by one
      out.pool_id[r] = find_or_add(out.hash[r], std::move(serial));
    }
  }
  return out;
}

}  // namespace xg
