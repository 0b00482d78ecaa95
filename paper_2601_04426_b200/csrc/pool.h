// Cross-grammar cache pool (Section 3.3): rule automata are keyed by a structural hash
// (Algorithm 1; cycles as in Algorithm 2) and verified against their canonical serialisation,
// so identical sub-structures are classified once and shared between grammars.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>
#include <map>
#include <memory>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "device_types.h"
#include "frontend.h"

namespace xg {

struct PoolRule {
  std::vector<uint64_t> serial;      // canonical serialisation (the exact identity of the rule)
  uint64_t hash = 0;
  bool built = false;                // at least one entry of this rule is in the pool
  std::vector<int> chunks;           // device chunks that hold this rule's entries
  std::vector<char> have;            // by canonical state index: the entry is in the pool (a just-in-time
                                     // grammar adds the entries of a rule one visited state at a time)
  std::vector<EntryDev> entries;     // by canonical state index
  std::vector<int2> counts;          // (accepted, uncertain) by canonical state index
};

// How one grammar's rules map onto the pool.
struct RuleInterning {
  std::vector<int> pool_id;                 // rule -> pool rule
  std::vector<std::vector<int>> canon;      // rule -> canonical index -> state offset inside the rule
  std::vector<uint64_t> hash;               // rule -> structural hash
};

// Hashes and canonical state orders only (no pool): Algorithm 1 bottom-up over the reference
// graph, Algorithm 2's refinement on cycles.
RuleInterning structural_hashes(const FlatGrammar& g);
// The pool-independent part of CachePool::intern (rule shapes, canonical orders, hashes): needs no lock, so
// threads that compile side by side only take turns for the pool lookups and the cache build.
std::shared_ptr<const void> prepare_interning(const FlatGrammar& g);

// Device memory in slabs with a first-fit free list.  Compiling a grammar needs a handful of
// device buffers (its tables, a batch of cache entries, its narrowed check lists); taking each
// from the driver costs a driver allocation apiece, which on a busy host takes from tens of
// microseconds to tens of milliseconds.  Slabs grow geometrically up to 256 MiB, so a pool that
// serves many grammars asks the driver a few dozen times in its life.  Not thread-safe: the
// owner serialises calls.
class DeviceArena {
 public:
  ~DeviceArena();
  void* alloc(size_t bytes);            // 256-byte aligned; nullptr when the device is out of memory
  void free(void* p);                   // p from alloc(); an empty slab goes back to the driver (unless it was reserved)
  bool reserve(size_t bytes);           // take slabs for `bytes` from the driver now; they stay until the arena is destroyed
  size_t reserved() const { return reserved_; }
 private:
  struct Slab { char* base = nullptr; size_t bytes = 0, used = 0; bool keep = false; std::map<size_t, size_t> free_blocks; };   // offset -> length
  std::vector<Slab> slabs_;
  std::unordered_map<void*, std::pair<int, size_t>> live_;      // block -> (slab, bytes)
  size_t reserved_ = 0;
};

class CachePool {
 public:
  explicit CachePool(const void* owner) : owner_(owner) {}
  ~CachePool();
  const void* owner() const { return owner_; }
  std::mutex mu;                            // one compile at a time per pool

  // find-or-create pool rules for every rule of `g`, callees first (call with `mu` held)
  // `prepared` (optional): the result of prepare_interning(g), computed without the lock
  RuleInterning intern(const FlatGrammar& g, const std::shared_ptr<const void>& prepared = nullptr);
  PoolRule& rule(int id) { return rules_[id]; }
  size_t n_rules() const { return rules_.size(); }
  // Device memory for one batch of freshly built entries.  Chunks are the unit of eviction
  // (Section 3.3 bounds the cross-grammar cache by a size limit with least-recently-used
  // eviction): a chunk may go once no live grammar uses any entry in it.
  void* allocate_device(size_t bytes, int* chunk_id);
  // Plain device memory from the pool's slabs for a grammar's own tables (not subject to the limit).
  void* allocate_plain(size_t bytes) { return arena_.alloc(bytes); }
  void free_plain(void* p) { if (p) arena_.free(p); }
  bool reserve(size_t bytes) { return arena_.reserve(bytes); }
  void retain(const std::vector<int>& chunk_ids);          // a grammar starts using these chunks
  void release(const std::vector<int>& chunk_ids);         // ... and stops (locks `mu` itself)
  void release_held(const std::vector<int>& chunk_ids);    // the same with `mu` already held
  void set_limit(long long bytes) { limit_ = bytes; }
  void enforce_limit();                                      // evict least recently used idle chunks (call with `mu` held)
  void note_rule_in_chunk(int rule_id, int chunk_id) { chunks_[chunk_id].rules.push_back(rule_id); }
  struct Stats { long long bytes = 0, reserved = 0, evicted_chunks = 0, evicted_bytes = 0; int live_rules = 0, chunks = 0; };
  Stats stats() const;
  // reusable build scratch (grow-only, one buffer per slot; call with `mu` held)
  void* scratch(int slot, size_t bytes);
  // reusable pinned host staging for uploads (grow-only, one buffer per slot; call with `mu` held).  A copy from
  // pageable memory makes the runtime synchronise the stream first; from here it is only enqueued.  The caller
  // must have synchronised with the previous copy out of a slot before writing to it again.
  void* pinned(int slot, size_t bytes);

  // Arena of the just-in-time builds (Section 3.5).  A build that runs inside the decode loop
  // cannot stop to learn its size on the host, so it takes its space on the device: a counter of
  // words used, bumped by the build itself.  One chunk at a time; when a build does not fit, the
  // host opens a larger one and the build is repeated.
  struct JitArena { uint32_t* base = nullptr; long long cap_words = 0; unsigned long long* d_used = nullptr; int chunk = -1; };
  // the current arena, or a fresh one of at least `min_words` when there is none or `renew` is set (call with `mu` held)
  // `first_words` > 0 sizes the very first arena (default 8 Mi words)
  const JitArena* jit_arena(long long min_words, bool renew, long long first_words = 0);
  // two events for timing a build step on the device (created on first use; nullptr if that fails)
  cudaEvent_t* timing_events();
  // host-side state of the just-in-time service (owned here, defined by the API layer)
  void* jit_host = nullptr;
  void (*jit_host_free)(void*) = nullptr;

 private:
  const void* owner_;
  std::vector<PoolRule> rules_;
  std::unordered_map<uint64_t, std::vector<int>> by_hash_;
  struct Chunk { void* ptr = nullptr; size_t bytes = 0; int refs = 0; uint64_t last_use = 0; std::vector<int> rules; };
  std::vector<Chunk> chunks_;
  DeviceArena arena_;
  long long limit_ = 0, bytes_ = 0, evicted_chunks_ = 0, evicted_bytes_ = 0;
  uint64_t clock_ = 0;
  std::vector<std::pair<void*, size_t>> scratch_, pinned_;
  JitArena jit_;
  cudaEvent_t timing_[2] = {nullptr, nullptr};
  int find_or_add(uint64_t hash, std::vector<uint64_t>&& serial);
};

// The order-sensitive hash of Algorithm 1 (the paper leaves it open; this is a 64-bit
// multiply-xorshift fold).
uint64_t hash_fold(uint64_t h, uint64_t x);

}  // namespace xg
