// C ABI of the token-mask library: argument checking, device memory, launches.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <chrono>
#include <cstring>
#include <map>
#include <memory>
#include <mutex>
#include <string>
#include <vector>

#include "device_types.h"
#include "frontend.h"
#include "kernels.cuh"
#include "pool.h"
#include "xg.h"

using namespace xg;

namespace {

thread_local std::string g_last_error;

xg_status_t set_error(xg_status_t st, const std::string& msg) {
  g_last_error = msg;
  return st;
}

#define XG_CUDA(expr)                                                                               \
  do {                                                                                              \
    cudaError_t err__ = (expr);                                                                     \
    if (err__ != cudaSuccess)                                                                       \
      return set_error(XG_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(err__));         \
  } while (0)

template <typename T>
T* device_copy(const std::vector<T>& v, cudaError_t* err) {
  T* p = nullptr;
  size_t bytes = std::max<size_t>(v.size(), 1) * sizeof(T);
  *err = cudaMalloc(&p, bytes);
  if (*err != cudaSuccess) return nullptr;
  if (!v.empty()) *err = cudaMemcpy(p, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice);
  return p;
}

// launch with programmatic stream serialisation (see step_kernel_prologue in kernels.cuh)
template <typename... KArgs, typename... Args>
cudaError_t launch_step_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, int cluster_x, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attrs[2];
  int n = 0;
  attrs[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x > 1) {
    attrs[n].id = cudaLaunchAttributeClusterDimension;
    attrs[n].val.clusterDim.x = cluster_x; attrs[n].val.clusterDim.y = 1; attrs[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attrs;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// a named range around every entry point that does device work, for timelines (costs nothing without a profiler)
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};

double now_ms() {
  return std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

}  // namespace

// Device arrays of matcher pointers, one per batch composition.  A decode loop calls with the same list of
// matchers step after step, or with one that differs in a request or two (continuous batching): the list is looked
// up among the cached compositions; a new one takes the least recently used entry and is uploaded with one
// asynchronous copy from the entry's own pinned staging buffer on the caller's stream.  After the tables have grown
// to the largest batch in use there is no allocation, no device-wide synchronisation and no blocking copy.
constexpr int kBatchEntries = 64;
constexpr int kDefaultRepeatThreshold = 64;
constexpr int kShareEntriesFromRepeat = 24;   // explicit states share cache entries (state classes) in grammars with an expanded repetition this long   // bounded repetitions of at least this many iterations are counted, not expanded
struct BatchSlot {
  std::vector<xg_matcher_t*> key;
  MatcherDev** dev_matchers = nullptr;   // [cap], inside the tokenizer's slab
  MatcherDev** staging = nullptr;        // [cap], pinned host memory
  cudaEvent_t uploaded = nullptr;        // the last upload from `staging` (an entry is reused only after it)
  bool upload_recorded = false;
  bool in_graph = false;                 // uploaded inside a stream capture: the graph's copy node reads `staging` at
                                         // every replay, so the entry is never reused
  int32_t* status = nullptr;             // [cap] scratch words of the two-kernel fill (shared by all entries)
  int32_t* done_count = nullptr;
  uint64_t last_use = 0;
};
struct BatchTables {
  int cap = 0;                           // requests per entry
  MatcherDev** dev_slab = nullptr;       // [kBatchEntries][cap]
  MatcherDev** host_slab = nullptr;      // pinned, same shape
  int32_t* words = nullptr;              // status[cap], done_count[cap]
  std::vector<BatchSlot> slots;
};

struct xg_tokenizer {
  VocabDev dev{};
  std::vector<void*> allocations;
  std::vector<int32_t> rank_to_id, id_to_rank;
  std::vector<uint32_t> first_rank;       // [257] host copy of VocabDev::first_rank
  int32_t vocab_size = 0, n_words = 0;
  int64_t first_byte_count[256] = {};     // tokens (other than EOS / special / empty) by first byte
  mutable std::mutex mu;
  mutable BatchTables batches;
  mutable uint64_t use_counter = 0;
};

// Host side of the just-in-time cache build (Section 3.5).  The cycle belongs to the pool: a snapshot of
// the pool's miss ring is copied to pinned memory; once it has arrived, the reported states are served from
// the pool or their builds are enqueued, grammar by grammar; once the builds' results have arrived, they are
// recorded and the cycle restarts.  One snapshot and one event per step, however many grammars decode.
constexpr int kJitBatchMax = 64;          // entries per build (one grammar, one set of launches)
constexpr int kJitCycleEntries = 512;     // entries per cycle, over all grammars
constexpr int kJitCycleBuilds = 128;      // builds per cycle
struct JitHostResult {                    // pinned; written by asynchronous copies
  JitRing ring;
  EntryDev entries[kJitCycleEntries];
  int2 counts[kJitCycleEntries];
  int result[kJitCycleBuilds][2];
  long long total_words[kJitCycleBuilds];
};
struct JitFlight {                        // one enqueued build
  xg_grammar* g;
  std::vector<int32_t> reps;
  int chunk, entry_offset, index;
};
struct JitPool {
  JitRing* d_ring = nullptr;
  JitHostResult* h = nullptr;
  cudaEvent_t ev = nullptr;
  int phase = 0;                          // 0 idle, 1 snapshot on its way, 2 builds on their way
  uint32_t ring_seen = 0;
  std::vector<xg_grammar*> slots;         // the pool's just-in-time grammars by slot (nullptr once destroyed)
  std::vector<JitFlight> flights;
};
struct JitState {                         // per grammar
  bool enabled = false;
  int slot = -1;
  std::vector<int32_t> rep;                    // state -> class representative
  std::vector<int32_t> member_begin, members;  // representative -> the states of its class (CSR over all states)
  std::vector<uint8_t> status;                 // per representative: 0 missing, 1 build in flight, 2 built
  int32_t* d_rep = nullptr;
  int32_t* d_pub_state = nullptr;              // [kJitBatchMax] staging of pool hits
  EntryDev* d_pub_entry = nullptr;
  RuleInterning in;
  std::vector<int> canon_of, rule_first;
  int n_built = 0, n_pool_hits = 0, n_missing = 0, n_in_flight = 0;
};

struct xg_grammar {
  const xg_tokenizer* tok = nullptr;
  std::shared_ptr<CachePool> pool;
  FlatGrammar flat;                     // what the device runs on: with counted repetitions, one state record per class of counts
  FlatGrammar base;                     // the automata as the front end made them (only kept when they differ from `flat`)
  bool counted = false;                 // the grammar has counted repetitions (Section 3.6): `base` is set
  const FlatGrammar& tables() const { return counted ? base : flat; }
  std::vector<EntryDev> entries;        // [n_states], host copy of the device headers
  std::vector<int2> entry_counts;       // [n_states] (accepted, uncertain)
  GrammarDev host_view{};               // device pointers
  GrammarDev* dev = nullptr;            // the same struct in device memory
  void* blob = nullptr;
  void* lookahead_arena = nullptr;      // this grammar's narrowed check lists
  size_t entries_offset = 0;            // where the entry headers sit inside `blob`
  std::vector<int> entry_chunk;         // [n_states] pool chunk that holds the state's entry (-1: none)
  std::vector<int> chunk_refs;          // pool chunks this grammar keeps alive
  xg_grammar_stats_t stats{};
  bool count_visits = false;            // add up the bytes the classification walks consume (statistics only)
  int max_check = 0;                    // longest check list of this grammar's entries (which fill kernel a batch gets)
  JitState jit;
  // buffers behind xg_grammar_get_cache_entry's view
  mutable std::vector<int32_t> view_list, view_unc;
  mutable std::vector<uint32_t> view_bits;
};

struct xg_cache_pool {
  std::shared_ptr<CachePool> impl;
};

struct xg_matcher {
  const xg_grammar* grammar = nullptr;
  MatcherDev* dev = nullptr;
  void* block = nullptr;
};

extern "C" {

const char* xg_last_error(void) { return g_last_error.c_str(); }

// ---------------------------------------------------------------------------------------------
// vocabulary: sort by bytes (trie order), upload
// ---------------------------------------------------------------------------------------------
xg_status_t xg_tokenizer_create(const uint8_t* bytes, const int64_t* offsets, int32_t vocab_size, int32_t eos_token_id,
                                const int32_t* special_ids, int32_t n_special, void* stream, xg_tokenizer_t** out) {
  NvtxRange nvtx_range("xg_tokenizer_create");
  (void)stream;
  if (!out) return set_error(XG_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (!offsets || vocab_size <= 0 || (!bytes && offsets[vocab_size] > 0)) return set_error(XG_ERR_INVALID_ARG, "bad vocabulary arrays");
  if (eos_token_id >= vocab_size || eos_token_id < -1) return set_error(XG_ERR_INVALID_ARG, "eos_token_id out of range");
  if (n_special < 0 || (n_special > 0 && !special_ids)) return set_error(XG_ERR_INVALID_ARG, "bad special_ids");
  int max_len = 0;
  for (int i = 0; i < vocab_size; ++i) {
    int64_t len = offsets[i + 1] - offsets[i];
    if (len < 0) return set_error(XG_ERR_INVALID_ARG, "offsets must be non-decreasing");
    if (len > kSlowMaxBytes) return set_error(XG_ERR_UNSUPPORTED, "tokens longer than 255 bytes are not supported");
    max_len = std::max<int>(max_len, (int)len);
  }
  std::vector<char> never(vocab_size, 0);
  for (int i = 0; i < n_special; ++i) {
    if (special_ids[i] < 0 || special_ids[i] >= vocab_size) return set_error(XG_ERR_INVALID_ARG, "special id out of range");
    never[special_ids[i]] = 1;
  }
  if (eos_token_id >= 0) never[eos_token_id] = 1;
  std::unique_ptr<xg_tokenizer> t(new xg_tokenizer());
  t->vocab_size = vocab_size;
  t->n_words = (vocab_size + 31) / 32;
  std::vector<int32_t>& order = t->rank_to_id;
  order.resize(vocab_size);
  for (int i = 0; i < vocab_size; ++i) order[i] = i;
  std::sort(order.begin(), order.end(), [&](int a, int b) {
    size_t la = (size_t)(offsets[a + 1] - offsets[a]), lb = (size_t)(offsets[b + 1] - offsets[b]);
    int c = std::min(la, lb) ? std::memcmp(bytes + offsets[a], bytes + offsets[b], std::min(la, lb)) : 0;
    if (c != 0) return c < 0;
    if (la != lb) return la < lb;
    return a < b;
  });
  t->id_to_rank.resize(vocab_size);
  std::vector<uint8_t> arena;
  std::vector<uint32_t> off(vocab_size + 1, 0);
  std::vector<uint8_t> never_rank(vocab_size, 0);
  arena.reserve((size_t)offsets[vocab_size] + 16);
  for (int r = 0; r < vocab_size; ++r) {
    int id = order[r];
    t->id_to_rank[id] = r;
    if (offsets[id + 1] > offsets[id]) arena.insert(arena.end(), bytes + offsets[id], bytes + offsets[id + 1]);
    off[r + 1] = (uint32_t)arena.size();
    never_rank[r] = (never[id] || offsets[id + 1] == offsets[id]) ? 1 : 0;
    if (!never_rank[r]) ++t->first_byte_count[bytes[offsets[id]]];
  }
  arena.resize(arena.size() + 16, 0);
  cudaError_t err = cudaSuccess;
  auto keep = [&](auto* p) { if (p) t->allocations.push_back((void*)p); return p; };
  t->dev.vocab_size = vocab_size;
  t->dev.n_words = t->n_words;
  t->dev.eos_id = eos_token_id;
  t->dev.max_len = max_len;
  t->dev.n_bytes = (uint32_t)arena.size();
  t->dev.pad = 0;
  t->dev.bytes = keep(device_copy(arena, &err));
  if (err == cudaSuccess) t->dev.offset = keep(device_copy(off, &err));
  if (err == cudaSuccess) t->dev.rank_to_id = keep(device_copy(t->rank_to_id, &err));
  if (err == cudaSuccess) t->dev.id_to_rank = keep(device_copy(t->id_to_rank, &err));
  if (err == cudaSuccess) t->dev.never = keep(device_copy(never_rank, &err));
  // in trie order the tokens that start with byte b are one run of ranks
  t->first_rank.assign(257, (uint32_t)vocab_size);
  for (int r = vocab_size - 1; r >= 0; --r)
    if (off[r + 1] > off[r]) t->first_rank[arena[off[r]]] = (uint32_t)r;
  for (int b2 = 255; b2 >= 0; --b2) t->first_rank[b2] = std::min(t->first_rank[b2], t->first_rank[b2 + 1]);
  if (err == cudaSuccess) t->dev.first_rank = keep(device_copy(t->first_rank, &err));
  if (err != cudaSuccess) {
    for (void* p : t->allocations) cudaFree(p);
    return set_error(XG_ERR_CUDA, std::string("vocabulary upload: ") + cudaGetErrorString(err));
  }
  *out = t.release();
  return XG_OK;
}

void xg_tokenizer_destroy(xg_tokenizer_t* t) {
  if (!t) return;
  for (auto& s : t->batches.slots) if (s.uploaded) cudaEventDestroy(s.uploaded);
  cudaFree(t->batches.dev_slab); cudaFree(t->batches.words);
  if (t->batches.host_slab) cudaFreeHost(t->batches.host_slab);
  for (void* p : t->allocations) cudaFree(p);
  delete t;
}

// ---------------------------------------------------------------------------------------------
// bounds-checking build
// ---------------------------------------------------------------------------------------------
int32_t xg_debug_bounds_enabled(void) {
#ifdef XG_DEBUG_BOUNDS
  return 1;
#else
  return 0;
#endif
}

xg_status_t xg_debug_bounds_check(void* stream) {
#ifdef XG_DEBUG_BOUNDS
  static const char* what_name[] = {"?", "automaton state", "scan edge", "wait edge", "gather entry", "byte class", "token rank", "token bytes",
                                    "chart set", "chart item", "walk item", "plan entry", "mask row word", "cluster block", "check list entry", "cache entry"};
  XG_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  unsigned long long word = 0, zero = 0;
  XG_CUDA(cudaMemcpyFromSymbol(&word, g_bounds_violation, sizeof word));
  if (!word) return XG_OK;
  XG_CUDA(cudaMemcpyToSymbol(g_bounds_violation, &zero, sizeof zero));
  const int what = (int)((word >> 48) & 0x7FFF);
  return set_error(XG_ERR_BOUNDS, std::string("bounds violation in a kernel: ") + (what >= 1 && what <= 15 ? what_name[what] : "?") + " index " +
                                      std::to_string((long long)((word >> 24) & 0xFFFFFF)) + " (low 24 bits), limit " + std::to_string((long long)(word & 0xFFFFFF)));
#else
  (void)stream;
  return XG_OK;
#endif
}

xg_status_t xg_cache_pool_create(const xg_tokenizer_t* tok, xg_cache_pool_t** out) {
  if (!tok || !out) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  *out = new xg_cache_pool{std::make_shared<CachePool>((const void*)tok)};
  return XG_OK;
}
void xg_cache_pool_destroy(xg_cache_pool_t* pool) { delete pool; }

xg_status_t xg_cache_pool_set_limit(xg_cache_pool_t* pool, int64_t max_bytes) {
  if (!pool) return set_error(XG_ERR_INVALID_ARG, "NULL pool");
  std::lock_guard<std::mutex> lock(pool->impl->mu);
  pool->impl->set_limit(max_bytes);
  pool->impl->enforce_limit();
  return XG_OK;
}

xg_status_t xg_cache_pool_reserve(xg_cache_pool_t* pool, int64_t bytes) {
  if (!pool || bytes < 0) return set_error(XG_ERR_INVALID_ARG, "bad argument");
  std::lock_guard<std::mutex> lock(pool->impl->mu);
  if (!pool->impl->reserve((size_t)bytes)) return set_error(XG_ERR_OOM, "the device has no room for the reservation");
  return XG_OK;
}

xg_status_t xg_cache_pool_stats(xg_cache_pool_t* pool, xg_cache_pool_stats_t* out) {
  if (!pool || !out) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  std::lock_guard<std::mutex> lock(pool->impl->mu);
  const CachePool::Stats s = pool->impl->stats();
  out->bytes = s.bytes; out->reserved_bytes = s.reserved; out->evicted_bytes = s.evicted_bytes; out->evicted_chunks = s.evicted_chunks;
  out->live_rules = s.live_rules; out->chunks = s.chunks;
  return XG_OK;
}

// ---------------------------------------------------------------------------------------------
// grammar compilation
// ---------------------------------------------------------------------------------------------
// the entry headers alone, once the tables are on the device (the headers change twice during a compile: when the
// entries are built, and when this grammar's lookahead has narrowed their check lists)
static xg_status_t upload_entry_headers(xg_grammar* g, cudaStream_t stream) {
  if (!g->blob) return set_error(XG_ERR_INVALID_ARG, "internal: tables not uploaded yet");
  const size_t bytes = g->entries.size() * sizeof(EntryDev);
  void* stage = g->pool->pinned(1, bytes);            // (the caller synchronises between two uploads of the headers)
  if (!stage) return set_error(XG_ERR_OOM, "pinned staging allocation failed");
  std::memcpy(stage, g->entries.data(), bytes);
  XG_CUDA(cudaMemcpyAsync((uint8_t*)g->blob + g->entries_offset, stage, bytes, cudaMemcpyHostToDevice, stream));
  return XG_OK;
}

static xg_status_t upload_grammar(xg_grammar* g, cudaStream_t stream) {
  const FlatGrammar& f = g->flat;
  // one blob, sections 16-byte aligned
  size_t total = 0;
  auto reserve = [&](size_t bytes) { size_t at = total; total += (bytes + 15) & ~size_t(15); return at; };
  // classes of exactly one byte are encoded in place (no bitset lookup on the device)
  std::vector<uint32_t> class_code(f.n_classes);
  for (int c = 0; c < f.n_classes; ++c) {
    int count = 0, byte = 0;
    for (int b = 0; b < 256; ++b) if ((f.class_bits[(size_t)c * 8 + (b >> 5)] >> (b & 31)) & 1u) { ++count; byte = b; }
    class_code[c] = count == 1 ? (kLiteral | (uint32_t)byte) : (uint32_t)c;
  }
  std::vector<uint2> scan(f.scan_class.size()), wait(f.wait_rule.size());
  for (size_t e = 0; e < scan.size(); ++e) scan[e] = make_uint2(class_code[f.scan_class[e]], f.scan_target[e]);
  for (size_t e = 0; e < wait.size(); ++e) wait[e] = make_uint2(f.wait_rule[e], f.wait_target[e]);
  std::vector<StateRec> recs(f.n_states);
  for (int s = 0; s < f.n_states; ++s) {
    StateRec& r = recs[s];
    const int n_own = f.scan_own_end[s] - f.scan_begin[s], n_scan = f.scan_begin[s + 1] - f.scan_begin[s];
    const int n_wait = f.wait_begin[s + 1] - f.wait_begin[s], n_gather = f.gather_begin[s + 1] - f.gather_begin[s];
    if (n_scan > 65535 || n_wait > 65535 || n_gather > 65535) return set_error(XG_ERR_CAPACITY, "a state predicts more than 65535 edges");
    r.scan_begin = f.scan_begin[s]; r.n_own_n_scan = (uint32_t)n_own | ((uint32_t)n_scan << 16);
    r.wait_begin = f.wait_begin[s]; r.n_wait_n_gather = (uint32_t)n_wait | ((uint32_t)n_gather << 16);
    r.gather_begin = f.gather_begin[s];
    r.info = (uint32_t)f.state_rule[s] | (f.state_final[s] ? 0x80000000u : 0u);
    r.edge0_class = n_scan ? scan[f.scan_begin[s]].x : 0; r.edge0_target = n_scan ? scan[f.scan_begin[s]].y : 0;
  }
  const std::vector<uint32_t>& state_first = f.state_first;
  std::vector<int4> rep_state(f.rep_rec_base.size());
  for (size_t i = 0; i < rep_state.size(); ++i) rep_state[i] = make_int4(f.rep_rec_base[i], f.rep_lo[i], f.rep_hi[i], 0);
  size_t o_rep = reserve(rep_state.size() * sizeof(int4)), o_word = reserve(f.rec_word.size() * 4);
  size_t o_first = reserve(state_first.size() * 4), o_follow = reserve(f.rule_follow.size() * 4);
  size_t o_rec = reserve(recs.size() * sizeof(StateRec)), o_scan = reserve(scan.size() * sizeof(uint2)), o_wait = reserve(wait.size() * sizeof(uint2)),
         o_gs = reserve(f.gather_state.size() * 4), o_cb = reserve(f.class_bits.size() * 4),
         o_en = reserve((size_t)f.n_states * sizeof(EntryDev)), o_self = reserve(sizeof(GrammarDev));
  uint8_t* host = (uint8_t*)g->pool->pinned(0, total);       // (every compile ends with a synchronisation: the slot is free again)
  if (!host) return set_error(XG_ERR_OOM, "pinned staging allocation failed");
  std::memset(host, 0, total);
  auto put = [&](size_t at, const void* src, size_t bytes) { if (bytes) std::memcpy(host + at, src, bytes); };
  put(o_rep, rep_state.data(), rep_state.size() * sizeof(int4));
  put(o_word, f.rec_word.data(), f.rec_word.size() * 4);
  put(o_first, state_first.data(), state_first.size() * 4);
  put(o_follow, f.rule_follow.data(), f.rule_follow.size() * 4);
  put(o_rec, recs.data(), recs.size() * sizeof(StateRec));
  put(o_scan, scan.data(), scan.size() * sizeof(uint2));
  put(o_wait, wait.data(), wait.size() * sizeof(uint2));
  put(o_gs, f.gather_state.data(), f.gather_state.size() * 4);
  put(o_cb, f.class_bits.data(), f.class_bits.size() * 4);
  put(o_en, g->entries.data(), g->entries.size() * sizeof(EntryDev));
  if (!g->blob) {                        // from the pool's slabs (the caller holds the pool's lock)
    g->blob = g->pool->allocate_plain(total);
    if (!g->blob) return set_error(XG_ERR_OOM, "grammar table allocation failed");
  }
  uint8_t* d = (uint8_t*)g->blob;
  GrammarDev& v = g->host_view;
  v.n_states = f.n_states; v.n_rules = f.n_rules; v.n_classes = f.n_classes;
  v.root_rule = f.root_rule; v.root_nullable = f.root_nullable; v.root_start = f.rule_start[f.root_rule];
  v.state = (const StateRec*)(d + o_rec);
  v.scan_edge = (const uint2*)(d + o_scan);
  v.wait_edge = (const uint2*)(d + o_wait);
  v.gather_state = (const int32_t*)(d + o_gs);
  v.class_bits = (const uint32_t*)(d + o_cb);
  v.state_first = (const uint32_t*)(d + o_first);
  v.rule_follow = (const uint32_t*)(d + o_follow);
  v.entries = (const EntryDev*)(d + o_en);
  g->entries_offset = o_en;
  v.miss_ring = g->jit.slot >= 0 ? ((JitPool*)g->pool->jit_host)->d_ring : nullptr;
  v.jit_slot = g->jit.slot;
  v.rep_first = f.rep_first; v.rep_shift = f.rep_shift; v.rep_depth = f.rep_depth;
  v.n_words_states = f.rep_rec_base.empty() ? f.n_states : f.n_base_states;
  v.rep_state = rep_state.empty() ? nullptr : (const int4*)(d + o_rep);
  v.rec_word = f.rec_word.empty() ? nullptr : (const uint32_t*)(d + o_word);
  v.n_scan_edges = (int32_t)scan.size(); v.n_wait_edges = (int32_t)wait.size(); v.n_gather = (int32_t)f.gather_state.size();
  put(o_self, &v, sizeof(GrammarDev));
  g->dev = (GrammarDev*)(d + o_self);
  XG_CUDA(cudaMemcpyAsync(g->blob, host, total, cudaMemcpyHostToDevice, stream));
  return XG_OK;
}

// The classification's work list for positions states[0 .. n): per position one block for every kClassifyChunk of
// the tokens whose first byte one of the state's own edges can take (see classify_kernel).
static void classify_work_list(const xg_grammar* g, const int32_t* states, int n, std::vector<int2>* work) {
  const FlatGrammar& f = g->flat;
  const std::vector<uint32_t>& first_rank = g->tok->first_rank;
  work->clear();
  for (int k = 0; k < n; ++k) {
    const int s = states[k];
    uint32_t own[8] = {};
    for (int e = f.cedge_begin[s]; e < f.cedge_begin[s + 1]; ++e)
      for (int w = 0; w < 8; ++w) own[w] |= f.class_bits[(size_t)f.cedge_class[e] * 8 + w];
    long long total = 0;
    for (int w = 0; w < 8; ++w)
      for (uint32_t bits = own[w]; bits; bits &= bits - 1) { const int b = 32 * w + __builtin_ctz(bits); total += first_rank[b + 1] - first_rank[b]; }
    for (long long c = 0; c * kClassifyChunk < total; ++c) work->push_back(make_int2(k, (int)c));
  }
}

// classify + pack the given states (device work of the compile stage); fills entries / counts
static xg_status_t build_entries(xg_grammar* g, const std::vector<int32_t>& states, cudaStream_t stream) {
  if (states.empty()) return XG_OK;
  const VocabDev& v = g->tok->dev;
  const int W = v.n_words, V = v.vocab_size;
  const size_t row_bytes = (size_t)W * 4;
  const size_t budget = size_t(768) << 20;                         // scratch rows per batch
  const int per_batch = (int)std::max<size_t>(1, std::min<size_t>(std::min<size_t>(states.size(), 65535), budget / (3 * row_bytes)));
  // build scratch lives in the pool and is reused by later compiles (no allocation per grammar)
  const int over_cap = 1 << 16;
  CachePool& pool = *g->pool;
  int32_t* d_pos = (int32_t*)pool.scratch(0, per_batch * sizeof(int32_t));
  int32_t* h_pos = (int32_t*)pool.pinned(4, per_batch * sizeof(int32_t));
  uint32_t* d_rows = (uint32_t*)pool.scratch(1, 3 * row_bytes * per_batch);
  int2* d_counts = (int2*)pool.scratch(2, per_batch * sizeof(int2));
  PackPlan* d_plan = (PackPlan*)pool.scratch(3, per_batch * sizeof(PackPlan));
  long long* d_total = (long long*)pool.scratch(4, sizeof(long long));
  EntryDev* d_entries = (EntryDev*)pool.scratch(5, per_batch * sizeof(EntryDev));
  int2* d_over = (int2*)pool.scratch(6, over_cap * sizeof(int2));
  int* d_over_count = (int*)pool.scratch(7, 2 * sizeof(int));
  if (!h_pos || !d_pos || !d_rows || !d_counts || !d_plan || !d_total || !d_entries || !d_over || !d_over_count)
    return set_error(XG_ERR_OOM, "cache build scratch allocation failed");
  auto cleanup = [&]() {};
#define XG_CUDA_C(expr) do { cudaError_t e__ = (expr); if (e__ != cudaSuccess) { cleanup(); return set_error(XG_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__)); } } while (0)
  for (size_t begin = 0; begin < states.size(); begin += per_batch) {
    const int n = (int)std::min<size_t>(per_batch, states.size() - begin);
    uint32_t* acc = d_rows;                                      // the three row sets back to back: one clearing call
    uint32_t* unc = d_rows + (size_t)n * W;
    uint32_t* unr = d_rows + 2 * (size_t)n * W;
    std::memcpy(h_pos, states.data() + begin, n * sizeof(int32_t));       // (the previous batch ended with a synchronisation)
    XG_CUDA_C(cudaMemcpyAsync(d_pos, h_pos, n * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    XG_CUDA_C(cudaMemsetAsync(acc, 0, 3 * row_bytes * n, stream));  // blocks with nothing to scan leave their part of the rows untouched
    XG_CUDA_C(cudaMemsetAsync(d_over_count, 0, 2 * sizeof(int), stream));
    std::vector<int2> work;
    classify_work_list(g, states.data() + begin, n, &work);
    const int grid = (int)work.size();
    int2* h_work = (int2*)pool.pinned(5, std::max<size_t>(work.size(), 1) * sizeof(int2));
    int2* d_work = (int2*)pool.scratch(16, std::max<size_t>(work.size(), 1) * sizeof(int2));
    if (!h_work || !d_work) return set_error(XG_ERR_OOM, "cache build scratch allocation failed");
    if (grid > 0) {
      std::memcpy(h_work, work.data(), work.size() * sizeof(int2));
      XG_CUDA_C(cudaMemcpyAsync(d_work, h_work, work.size() * sizeof(int2), cudaMemcpyHostToDevice, stream));
    }
    cudaEvent_t* ev = pool.timing_events();            // device time of the classification itself, for the statistics
    if (ev) cudaEventRecord(ev[0], stream);
    if (g->count_visits) {
      unsigned long long* d_visits = (unsigned long long*)pool.scratch(8, sizeof(unsigned long long));
      if (!d_visits) return set_error(XG_ERR_OOM, "cache build scratch allocation failed");
      XG_CUDA_C(cudaMemsetAsync(d_visits, 0, sizeof(unsigned long long), stream));
      if (grid > 0) (g->counted ? classify_kernel<true, true> : classify_kernel<true, false>)<<<grid, 256, 0, stream>>>(g->host_view, v, d_pos, d_work, acc, unc, unr, d_over, d_over_count, over_cap, d_visits);
      unsigned long long visits = 0;
      XG_CUDA_C(cudaMemcpyAsync(&visits, d_visits, sizeof visits, cudaMemcpyDeviceToHost, stream));
      XG_CUDA_C(cudaStreamSynchronize(stream));
      g->stats.node_visits += (int64_t)visits;
    } else
    if (grid > 0) (g->counted ? classify_kernel<false, true> : classify_kernel<false, false>)<<<grid, 256, 0, stream>>>(g->host_view, v, d_pos, d_work, acc, unc, unr, d_over, d_over_count, over_cap, nullptr);
    XG_CUDA_C(cudaGetLastError());
    if (ev) cudaEventRecord(ev[1], stream);
    // count and plan are enqueued behind the classification at once; walks that left the fast path are rare, and when
    // there are some the two small kernels are simply run again after the exact fallback
    count_kernel<<<n, 256, 0, stream>>>(acc, unc, W, d_counts);
    plan_kernel<<<1, 1024, 0, stream>>>(d_counts, n, V, W, d_plan, d_total);
    XG_CUDA_C(cudaGetLastError());
    int over[2] = {0, 0};
    long long total_words = 0;
    XG_CUDA_C(cudaMemcpyAsync(over, d_over_count, 2 * sizeof(int), cudaMemcpyDeviceToHost, stream));
    XG_CUDA_C(cudaMemcpyAsync(&total_words, d_total, sizeof(long long), cudaMemcpyDeviceToHost, stream));
    XG_CUDA_C(cudaStreamSynchronize(stream));
    if (ev) { float ms = 0.f; if (cudaEventElapsedTime(&ms, ev[0], ev[1]) == cudaSuccess) g->stats.classify_ms += ms; }
    if (over[0] > over_cap) { cleanup(); return set_error(XG_ERR_CAPACITY, "too many token walks exceeded the fast path"); }
    for (int done = 0; done < over[0];) {          // exact fallback, a bounded number of pairs per round
      const int round = std::min(over[0] - done, 4096);
      // the exact walks' scratch comes from the pool too (grow-only, reused by later compiles)
      uint32_t* s_st = (uint32_t*)pool.scratch(9, (size_t)round * kSlowCap * 4);
      int32_t* s_org = (int32_t*)pool.scratch(10, (size_t)round * kSlowCap * 4);
      int32_t* s_lsb = (int32_t*)pool.scratch(14, (size_t)round * (kSlowMaxBytes + 2) * 4);
      if (!s_st || !s_org || !s_lsb) { cleanup(); return set_error(XG_ERR_OOM, "slow classification scratch allocation failed"); }
      classify_slow_kernel<<<(round + 63) / 64, 64, 0, stream>>>(g->host_view, v, d_pos, d_over + done, round, s_st, s_org, s_lsb, acc, unc, unr, d_over_count + 1);
      if (cudaStreamSynchronize(stream) != cudaSuccess) { cleanup(); return set_error(XG_ERR_CUDA, "slow classification failed"); }
      done += round;
    }
    if (over[0] > 0) {
      XG_CUDA_C(cudaMemcpy(over, d_over_count, 2 * sizeof(int), cudaMemcpyDeviceToHost));
      if (over[1]) { cleanup(); return set_error(XG_ERR_CAPACITY, "an Earley item set exceeded the supported size during cache build"); }
      count_kernel<<<n, 256, 0, stream>>>(acc, unc, W, d_counts);
      plan_kernel<<<1, 1024, 0, stream>>>(d_counts, n, V, W, d_plan, d_total);
      XG_CUDA_C(cudaGetLastError());
      XG_CUDA_C(cudaMemcpyAsync(&total_words, d_total, sizeof(long long), cudaMemcpyDeviceToHost, stream));
      XG_CUDA_C(cudaStreamSynchronize(stream));
    }
    int chunk_id = -1;
    uint32_t* arena = (uint32_t*)g->pool->allocate_device((size_t)std::max<long long>(total_words, 1) * 4, &chunk_id);
    if (!arena) { cleanup(); return set_error(XG_ERR_OOM, "cache arena allocation failed"); }
    pack_kernel<<<n, 256, 0, stream>>>(acc, unc, unr, d_plan, V, W, arena, d_entries, nullptr);
    (g->counted ? exit_kernel<true> : exit_kernel<false>)<<<n, 256, 0, stream>>>(g->host_view, v, d_pos, d_entries, nullptr);
    XG_CUDA_C(cudaGetLastError());
    std::vector<EntryDev> built(n);
    std::vector<int2> counts(n);
    XG_CUDA_C(cudaMemcpyAsync(built.data(), d_entries, n * sizeof(EntryDev), cudaMemcpyDeviceToHost, stream));
    XG_CUDA_C(cudaMemcpyAsync(counts.data(), d_counts, n * sizeof(int2), cudaMemcpyDeviceToHost, stream));
    XG_CUDA_C(cudaStreamSynchronize(stream));
    for (int k = 0; k < n; ++k) { g->entries[states[begin + k]] = built[k]; g->entry_counts[states[begin + k]] = counts[k]; g->entry_chunk[states[begin + k]] = chunk_id; }
  }
  cleanup();
#undef XG_CUDA_C
  return XG_OK;
}

// Lookahead pass (Section 3.3): the pool's entries are context-free; each grammar narrows their
// uncertain lists with its own follow sets.  Count, exclusive scan on the host (a few thousand
// numbers), compact.  The grammar's entry headers must already be on the device.
static xg_status_t narrow_check_lists(xg_grammar* g, const std::vector<int32_t>& scannable, const std::vector<int32_t>& rep, cudaStream_t stream, bool* narrowed) {
  *narrowed = false;
  std::vector<int32_t> states;
  for (int s : scannable) if (g->entries[s].n_unc > 0 && rep[s] == s) states.push_back(s);      // one list per shared entry
  if (states.empty()) return XG_OK;
  const int n = (int)states.size();
  if (n > 2000000) return set_error(XG_ERR_CAPACITY, "too many cache entries with uncertain tokens");
  CachePool& pool = *g->pool;
  int32_t* d_states = (int32_t*)pool.scratch(11, (size_t)n * 4);
  int32_t* d_counts = (int32_t*)pool.scratch(12, (size_t)n * 4);
  long long* d_offsets = (long long*)pool.scratch(13, (size_t)n * 8);
  if (!d_states || !d_counts || !d_offsets) return set_error(XG_ERR_OOM, "lookahead scratch allocation failed");
  int32_t* h_states = (int32_t*)pool.pinned(2, (size_t)n * 4);
  long long* h_offsets = (long long*)pool.pinned(3, (size_t)n * 8);
  if (!h_states || !h_offsets) return set_error(XG_ERR_OOM, "pinned staging allocation failed");
  std::memcpy(h_states, states.data(), (size_t)n * 4);
  XG_CUDA(cudaMemcpyAsync(d_states, h_states, (size_t)n * 4, cudaMemcpyHostToDevice, stream));
  lookahead_count_kernel<<<n, 256, 0, stream>>>(g->host_view, g->tok->dev, d_states, d_counts, nullptr);
  XG_CUDA(cudaGetLastError());
  std::vector<int32_t> counts(n);
  XG_CUDA(cudaMemcpyAsync(counts.data(), d_counts, (size_t)n * 4, cudaMemcpyDeviceToHost, stream));
  XG_CUDA(cudaStreamSynchronize(stream));
  std::vector<long long> offsets(n);
  long long total = 0;
  for (int k = 0; k < n; ++k) { offsets[k] = total; total += 3LL * counts[k]; }
  g->lookahead_arena = pool.allocate_plain((size_t)std::max<long long>(total, 1) * 4);
  if (!g->lookahead_arena) return set_error(XG_ERR_OOM, "check list allocation failed");
  std::memcpy(h_offsets, offsets.data(), (size_t)n * 8);
  XG_CUDA(cudaMemcpyAsync(d_offsets, h_offsets, (size_t)n * 8, cudaMemcpyHostToDevice, stream));
  lookahead_compact_kernel<<<n, 256, 0, stream>>>(g->host_view, g->tok->dev, d_states, d_offsets, d_counts, (uint32_t*)g->lookahead_arena, nullptr);
  XG_CUDA(cudaGetLastError());          // (the caller synchronises once the narrowed headers are on their way too)
  uint32_t* arena = (uint32_t*)g->lookahead_arena;
  for (int k = 0; k < n; ++k) {
    EntryDev& e = g->entries[states[k]];
    e.chk_rank = arena + offsets[k];
    e.chk_exit = e.chk_rank + counts[k];
    e.chk_info = e.chk_exit + counts[k];
    e.n_chk = counts[k];
  }
  for (int s : scannable) {
    if (rep[s] == s) continue;
    const EntryDev& r = g->entries[rep[s]];
    EntryDev& e = g->entries[s];
    e.chk_rank = r.chk_rank; e.chk_exit = r.chk_exit; e.chk_info = r.chk_info; e.n_chk = r.n_chk;
  }
  *narrowed = true;
  return XG_OK;
}

// ---------------------------------------------------------------------------------------------
// just-in-time cache build (Section 3.5)
// ---------------------------------------------------------------------------------------------
// device scratch of the just-in-time builds: the pool's, separate from the compile-time build's (which may be
// running on another stream) and sized once for a full batch, so it is never reallocated inside a decode loop
struct JitScratch {
  int32_t* pos; uint32_t* rows; int2* counts; PackPlan* plan; long long* total; EntryDev* entries; int2* over; int* over_count; int* result;
  int32_t* list_counts; long long* list_offsets; int* go_lists; int* one;
};
static bool jit_scratch(CachePool& pool, int W, JitScratch* sc) {
  const size_t row_bytes = (size_t)W * 4;
  sc->pos = (int32_t*)pool.scratch(20, kJitBatchMax * sizeof(int32_t));
  sc->rows = (uint32_t*)pool.scratch(21, 3 * row_bytes * kJitBatchMax);
  sc->counts = (int2*)pool.scratch(22, kJitBatchMax * sizeof(int2));
  sc->plan = (PackPlan*)pool.scratch(23, kJitBatchMax * sizeof(PackPlan));
  sc->total = (long long*)pool.scratch(24, sizeof(long long));
  sc->entries = (EntryDev*)pool.scratch(25, kJitBatchMax * sizeof(EntryDev));
  sc->over = (int2*)pool.scratch(26, 64 * sizeof(int2));
  sc->over_count = (int*)pool.scratch(27, 2 * sizeof(int));
  sc->result = (int*)pool.scratch(28, 2 * sizeof(int));
  sc->list_counts = (int32_t*)pool.scratch(29, kJitBatchMax * sizeof(int32_t));
  sc->list_offsets = (long long*)pool.scratch(30, kJitBatchMax * sizeof(long long));
  sc->go_lists = (int*)pool.scratch(31, sizeof(int));
  sc->one = (int*)pool.scratch(32, sizeof(int));            // holds 1 (set when a grammar registers)
  return sc->one && sc->list_counts && sc->list_offsets && sc->go_lists && sc->pos && sc->rows && sc->counts && sc->plan && sc->total && sc->entries && sc->over && sc->over_count && sc->result;
}

static void jit_pool_free(void* p) {
  JitPool* jp = (JitPool*)p;
  cudaFree(jp->d_ring);
  if (jp->h) cudaFreeHost(jp->h);
  if (jp->ev) cudaEventDestroy(jp->ev);
  delete jp;
}

// undo jit_allocate (call with the pool's lock held)
static void jit_release(xg_grammar* g) {
  cudaDeviceSynchronize();               // a build of this grammar may still be on its way
  if (g->pool) g->pool->free_plain(g->jit.d_rep);
  g->jit.d_rep = nullptr; g->jit.d_pub_state = nullptr; g->jit.d_pub_entry = nullptr;
  JitPool* jp = g->pool ? (JitPool*)g->pool->jit_host : nullptr;
  if (jp && g->jit.slot >= 0) {
    jp->slots[g->jit.slot] = nullptr;
    jp->flights.erase(std::remove_if(jp->flights.begin(), jp->flights.end(), [&](const JitFlight& fl) { return fl.g == g; }), jp->flights.end());
  }
  g->jit.slot = -1;
  g->jit.enabled = false;
}

// per-grammar device arrays, the pool's ring and scratch; registers the grammar in the pool (call with the pool's lock held)
static xg_status_t jit_allocate(xg_grammar* g, long long first_arena_words) {
  JitState& j = g->jit;
  CachePool& pool = *g->pool;
  JitScratch sc;
  if (!jit_scratch(pool, g->tok->n_words, &sc) || !pool.jit_arena(0, false, first_arena_words)) return set_error(XG_ERR_OOM, "just-in-time scratch allocation failed");
  const int one = 1;
  XG_CUDA(cudaMemcpy(sc.one, &one, sizeof(int), cudaMemcpyHostToDevice));
  if (!pool.jit_host) {
    JitPool* jp = new JitPool();
    pool.jit_host = jp;
    pool.jit_host_free = jit_pool_free;
    XG_CUDA(cudaMalloc(&jp->d_ring, sizeof(JitRing)));
    XG_CUDA(cudaMemset(jp->d_ring, 0, sizeof(JitRing)));
    XG_CUDA(cudaHostAlloc(&jp->h, sizeof(JitHostResult), cudaHostAllocDefault));
    std::memset(jp->h, 0, sizeof(JitHostResult));
    XG_CUDA(cudaEventCreateWithFlags(&jp->ev, cudaEventDisableTiming));
  }
  JitPool* jp = (JitPool*)pool.jit_host;
  if (!jp->d_ring || !jp->h || !jp->ev) return set_error(XG_ERR_CUDA, "the pool's just-in-time state is incomplete");
  // one block from the pool's slabs: [rep | staged states | staged entries]
  const size_t S = (size_t)std::max(g->flat.n_states, 1);
  const size_t o_state = (S * 4 + 255) & ~size_t(255), o_entry = o_state + 256;
  static_assert(kJitBatchMax * sizeof(int32_t) <= 256, "staging area too small");
  char* block = (char*)pool.allocate_plain(o_entry + kJitBatchMax * sizeof(EntryDev));
  if (!block) return set_error(XG_ERR_OOM, "just-in-time tables allocation failed");
  j.d_rep = (int32_t*)block;
  j.d_pub_state = (int32_t*)(block + o_state);
  j.d_pub_entry = (EntryDev*)(block + o_entry);
  for (size_t k = 0; k < jp->slots.size() && j.slot < 0; ++k) if (!jp->slots[k]) { jp->slots[k] = g; j.slot = (int)k; }
  if (j.slot < 0) { jp->slots.push_back(g); j.slot = (int)jp->slots.size() - 1; }
  return XG_OK;
}

// the host's record of entries that now exist on the device for the representatives `reps`:
// grammar copy for every class member, pool registration, chunk references
static void jit_record(xg_grammar* g, const std::vector<int32_t>& reps, const EntryDev* entries, const int2* counts, int chunk) {
  JitState& j = g->jit;
  const FlatGrammar& f = g->flat;
  CachePool& pool = *g->pool;
  for (size_t k = 0; k < reps.size(); ++k) {
    const int r = reps[k];
    const int rule = f.state_rule[r];
    PoolRule& pr = pool.rule(j.in.pool_id[rule]);
    const int n_local = (int)j.in.canon[rule].size();
    pr.entries.resize(n_local); pr.counts.resize(n_local); pr.have.resize(n_local, 0);
    for (int q = j.member_begin[r]; q < j.member_begin[r + 1]; ++q) {
      const int s = j.members[q];
      g->entries[s] = entries[k]; g->entry_counts[s] = counts[k]; g->entry_chunk[s] = chunk;
      g->max_check = std::max(g->max_check, (int)entries[k].n_unc);        // (its narrowed list is at most this long)
      const int c = j.canon_of[s];
      if (c >= 0 && !pr.have[c]) { pr.entries[c] = entries[k]; pr.counts[c] = counts[k]; pr.have[c] = 1; }
    }
    pr.built = true;
    if (chunk >= 0 && std::find(pr.chunks.begin(), pr.chunks.end(), chunk) == pr.chunks.end()) { pr.chunks.push_back(chunk); pool.note_rule_in_chunk(j.in.pool_id[rule], chunk); }
    if (j.status[r] != 2) { j.status[r] = 2; --j.n_missing; }
  }
  if (chunk >= 0 && std::find(g->chunk_refs.begin(), g->chunk_refs.end(), chunk) == g->chunk_refs.end()) {
    g->chunk_refs.push_back(chunk);
    pool.retain(std::vector<int>{chunk});
  }
}

// This grammar's lookahead narrows the check lists of the entries just published for `d_states` (only in its own
// device copy of the headers: the pool keeps them context-free).  `go`: device flag, the step is skipped when it is 0.
static void jit_enqueue_narrowing(xg_grammar* g, const JitScratch& sc, const CachePool::JitArena* arena, const int32_t* d_states, int n,
                                  const int* go, cudaStream_t stream) {
  EntryDev* dev_entries = const_cast<EntryDev*>(g->host_view.entries);
  lookahead_count_kernel<<<n, 256, 0, stream>>>(g->host_view, g->tok->dev, d_states, sc.list_counts, go);
  jit_reserve_lists_kernel<<<1, 32, 0, stream>>>(sc.list_counts, n, sc.list_offsets, arena->d_used, arena->cap_words, go, sc.go_lists);
  lookahead_compact_kernel<<<n, 256, 0, stream>>>(g->host_view, g->tok->dev, d_states, sc.list_offsets, sc.list_counts, arena->base, sc.go_lists);
  jit_patch_lists_kernel<<<(g->flat.n_states + 255) / 256, 256, 0, stream>>>(dev_entries, g->jit.d_rep, g->flat.n_states, d_states, sc.list_counts,
                                                                             sc.list_offsets, arena->base, n, sc.go_lists);
}

// publish host-side entry headers for `reps` (pool hits, or entries built by the synchronous path)
static xg_status_t jit_publish_from_host(xg_grammar* g, const std::vector<int32_t>& reps, const std::vector<EntryDev>& entries, cudaStream_t stream) {
  JitState& j = g->jit;
  for (size_t begin = 0; begin < reps.size(); begin += kJitBatchMax) {
    const int n = (int)std::min<size_t>(kJitBatchMax, reps.size() - begin);
    // pageable sources: the runtime stages them before these calls return
    XG_CUDA(cudaMemcpyAsync(j.d_pub_state, reps.data() + begin, n * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    XG_CUDA(cudaMemcpyAsync(j.d_pub_entry, entries.data() + begin, n * sizeof(EntryDev), cudaMemcpyHostToDevice, stream));
    jit_publish_kernel<<<(g->flat.n_states + 255) / 256, 256, 0, stream>>>(const_cast<EntryDev*>(g->host_view.entries), j.d_rep, g->flat.n_states,
                                                                           j.d_pub_state, j.d_pub_entry, n, nullptr);
    const CachePool::JitArena* arena = g->pool->jit_arena(0, false);
    JitScratch sc;
    if (arena && jit_scratch(*g->pool, g->tok->n_words, &sc)) {
      if (std::find(g->chunk_refs.begin(), g->chunk_refs.end(), arena->chunk) == g->chunk_refs.end()) {
        g->chunk_refs.push_back(arena->chunk);
        g->pool->retain(std::vector<int>{arena->chunk});
      }
      jit_enqueue_narrowing(g, sc, arena, j.d_pub_state, n, sc.one, stream);
    }
    XG_CUDA(cudaGetLastError());
  }
  return XG_OK;
}

// Enqueue the build of `reps` (at most kJitBatchMax, one grammar) without any host round trip; its
// results go to slice (`entry_offset`, `index`) of the pool's pinned result block.
static xg_status_t jit_enqueue_build(JitPool* jp, xg_grammar* g, const std::vector<int32_t>& reps, bool renew_arena, long long min_words,
                                     int entry_offset, int index, cudaStream_t stream) {
  JitState& j = g->jit;
  CachePool& pool = *g->pool;
  const VocabDev& v = g->tok->dev;
  const int W = v.n_words, V = v.vocab_size, n = (int)reps.size();
  const size_t row_bytes = (size_t)W * 4;
  const CachePool::JitArena* arena = pool.jit_arena(min_words, renew_arena);
  if (!arena) return set_error(XG_ERR_OOM, "just-in-time arena allocation failed");
  JitScratch sc;
  if (!jit_scratch(pool, W, &sc)) return set_error(XG_ERR_OOM, "just-in-time scratch allocation failed");
  if (std::find(g->chunk_refs.begin(), g->chunk_refs.end(), arena->chunk) == g->chunk_refs.end()) {     // in use from now on
    g->chunk_refs.push_back(arena->chunk);
    pool.retain(std::vector<int>{arena->chunk});
  }
  uint32_t* acc = sc.rows;
  uint32_t* unc = sc.rows + (size_t)kJitBatchMax * W;
  uint32_t* unr = sc.rows + 2 * (size_t)kJitBatchMax * W;
  XG_CUDA(cudaMemcpyAsync(sc.pos, reps.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
  XG_CUDA(cudaMemsetAsync(acc, 0, row_bytes * n, stream));
  XG_CUDA(cudaMemsetAsync(unc, 0, row_bytes * n, stream));
  XG_CUDA(cudaMemsetAsync(unr, 0, row_bytes * n, stream));
  XG_CUDA(cudaMemsetAsync(sc.over_count, 0, 2 * sizeof(int), stream));
  std::vector<int2> work;
  classify_work_list(g, reps.data(), n, &work);
  if (!work.empty()) {
    // (a pageable source: the runtime stages it before the call returns; a few hundred bytes)
    int2* d_work = (int2*)pool.scratch(33, work.size() * sizeof(int2));
    if (!d_work) return set_error(XG_ERR_OOM, "just-in-time scratch allocation failed");
    XG_CUDA(cudaMemcpyAsync(d_work, work.data(), work.size() * sizeof(int2), cudaMemcpyHostToDevice, stream));
    (g->counted ? classify_kernel<false, true> : classify_kernel<false, false>)<<<(int)work.size(), 256, 0, stream>>>(g->host_view, v, sc.pos, d_work, acc, unc, unr, sc.over, sc.over_count, 64, nullptr);
  }
  count_kernel<<<n, 256, 0, stream>>>(acc, unc, W, sc.counts);
  plan_kernel<<<1, 1024, 0, stream>>>(sc.counts, n, V, W, sc.plan, sc.total);
  jit_reserve_kernel<<<1, 32, 0, stream>>>(sc.plan, n, sc.total, arena->d_used, arena->cap_words, sc.over_count, sc.result);
  pack_kernel<<<n, 256, 0, stream>>>(acc, unc, unr, sc.plan, V, W, arena->base, sc.entries, sc.result);
  (g->counted ? exit_kernel<true> : exit_kernel<false>)<<<n, 256, 0, stream>>>(g->host_view, v, sc.pos, sc.entries, sc.result);
  jit_publish_kernel<<<(g->flat.n_states + 255) / 256, 256, 0, stream>>>(const_cast<EntryDev*>(g->host_view.entries), j.d_rep, g->flat.n_states,
                                                                         sc.pos, sc.entries, n, sc.result);
  jit_enqueue_narrowing(g, sc, arena, sc.pos, n, sc.result, stream);
  XG_CUDA(cudaGetLastError());
  // the scratch is reused by the next build in stream order: take the results out first
  XG_CUDA(cudaMemcpyAsync(jp->h->entries + entry_offset, sc.entries, n * sizeof(EntryDev), cudaMemcpyDeviceToHost, stream));
  XG_CUDA(cudaMemcpyAsync(jp->h->counts + entry_offset, sc.counts, n * sizeof(int2), cudaMemcpyDeviceToHost, stream));
  XG_CUDA(cudaMemcpyAsync(jp->h->result[index], sc.result, 2 * sizeof(int), cudaMemcpyDeviceToHost, stream));
  XG_CUDA(cudaMemcpyAsync(&jp->h->total_words[index], sc.total, sizeof(long long), cudaMemcpyDeviceToHost, stream));
  JitFlight fl;
  fl.g = g; fl.reps = reps; fl.chunk = arena->chunk; fl.entry_offset = entry_offset; fl.index = index;
  jp->flights.push_back(fl);
  for (int r : reps) j.status[r] = 1;
  j.n_in_flight += n;
  return XG_OK;
}

// One pool's cycle over the grammars in `eligible`.  *idle = true once a snapshot taken inside this
// call held nothing new and nothing is in flight (only reachable with wait).
static xg_status_t jit_advance(CachePool& pool, const std::vector<xg_grammar*>& eligible, cudaStream_t stream, bool wait, bool* idle) {
  JitPool* jp = (JitPool*)pool.jit_host;
  bool fresh = false;            // the snapshot being looked at was taken inside this call
  *idle = false;
  for (int guard = 0; guard < 100000; ++guard) {
    if (jp->phase == 0) {
      bool any_missing = false;
      for (xg_grammar* g : eligible) any_missing = any_missing || g->jit.n_missing > 0;
      if (!any_missing) { *idle = true; return XG_OK; }           // everything is built: nothing can be reported any more
      XG_CUDA(cudaMemcpyAsync(&jp->h->ring, jp->d_ring, sizeof(JitRing), cudaMemcpyDeviceToHost, stream));
      XG_CUDA(cudaEventRecord(jp->ev, stream));
      jp->phase = 1;
      fresh = true;
      if (!wait) return XG_OK;
      continue;
    }
    if (wait) XG_CUDA(cudaEventSynchronize(jp->ev));
    else {
      cudaError_t q = cudaEventQuery(jp->ev);
      if (q == cudaErrorNotReady) return XG_OK;
      if (q != cudaSuccess) return set_error(XG_ERR_CUDA, std::string("just-in-time event: ") + cudaGetErrorString(q));
    }
    if (jp->phase == 2) {                      // the builds have finished
      std::vector<JitFlight> flights;
      flights.swap(jp->flights);
      jp->phase = 0;
      std::vector<JitFlight> again;
      for (JitFlight& fl : flights) {
        xg_grammar* g = fl.g;
        g->jit.n_in_flight -= (int)fl.reps.size();
        const int* result = jp->h->result[fl.index];
        if (result[0] == 1) {
          jit_record(g, fl.reps, jp->h->entries + fl.entry_offset, jp->h->counts + fl.entry_offset, fl.chunk);
          g->jit.n_built += (int)fl.reps.size();
        } else if (result[1] == 1) {           // no room: the same states again, in a larger arena
          for (int r : fl.reps) g->jit.status[r] = 0;
          again.push_back(fl);
        } else {                               // a walk left the fast path: the exact build with its host round trips
          for (int r : fl.reps) g->jit.status[r] = 0;
          xg_status_t st = build_entries(g, fl.reps, stream);
          if (st != XG_OK) return st;
          std::vector<EntryDev> es;
          std::vector<int2> cs;
          for (int r : fl.reps) { es.push_back(g->entries[r]); cs.push_back(g->entry_counts[r]); }
          st = jit_publish_from_host(g, fl.reps, es, stream);
          if (st != XG_OK) return st;
          for (size_t k = 0; k < fl.reps.size(); ++k) jit_record(g, std::vector<int32_t>{fl.reps[k]}, &es[k], &cs[k], g->entry_chunk[fl.reps[k]]);
          g->jit.n_built += (int)fl.reps.size();
        }
      }
      if (!again.empty()) {
        long long need = 1 << 16;
        for (JitFlight& fl : again) need += jp->h->total_words[fl.index];
        bool renew = true;
        for (JitFlight& fl : again) {
          xg_status_t st = jit_enqueue_build(jp, fl.g, fl.reps, renew, need, fl.entry_offset, fl.index, stream);
          if (st != XG_OK) return st;
          renew = false;
        }
        XG_CUDA(cudaEventRecord(jp->ev, stream));
        jp->phase = 2;
        if (!wait) return XG_OK;
      }
      continue;
    }
    // phase 1: a snapshot of the miss ring has arrived
    jp->phase = 0;
    const uint32_t count = jp->h->ring.count;
    uint32_t from = jp->ring_seen;
    if (count - from > (uint32_t)kJitRingCap) from = count - kJitRingCap;
    std::vector<std::pair<xg_grammar*, std::vector<int32_t>>> want;      // in order of first report
    for (uint32_t i = from; i != count; ++i) {
      const int2 m = jp->h->ring.miss[i % kJitRingCap];
      if (m.x < 0 || m.x >= (int)jp->slots.size()) continue;
      xg_grammar* g = jp->slots[m.x];
      if (!g || std::find(eligible.begin(), eligible.end(), g) == eligible.end()) continue;
      if (m.y < 0 || m.y >= g->flat.n_states) continue;
      const int r = g->jit.rep[m.y];
      if (g->jit.status[r] != 0) continue;
      size_t w = 0;
      while (w < want.size() && want[w].first != g) ++w;
      if (w == want.size()) want.emplace_back(g, std::vector<int32_t>());
      if (std::find(want[w].second.begin(), want[w].second.end(), r) == want[w].second.end()) want[w].second.push_back(r);
    }
    jp->ring_seen = count;
    if (want.empty()) {
      if (wait && fresh) { *idle = true; return XG_OK; }
      continue;                                // take a fresh snapshot
    }
    fresh = false;
    int entry_offset = 0, index = 0;
    for (auto& gw : want) {
      xg_grammar* g = gw.first;
      JitState& j = g->jit;
      const FlatGrammar& f = g->flat;
      // cache hit (Section 3.5): the pool already holds the entry (another grammar has built it since)
      std::vector<int32_t> hit_reps, build_reps;
      std::vector<EntryDev> hit_entries;
      std::vector<int2> hit_counts;
      for (int r : gw.second) {
        const PoolRule& pr = pool.rule(j.in.pool_id[f.state_rule[r]]);
        const int c = j.canon_of[r];
        if (pr.built && c >= 0 && c < (int)pr.have.size() && pr.have[c]) {
          hit_reps.push_back(r); hit_entries.push_back(pr.entries[c]); hit_counts.push_back(pr.counts[c]);
          for (int ch : pr.chunks)
            if (std::find(g->chunk_refs.begin(), g->chunk_refs.end(), ch) == g->chunk_refs.end()) { g->chunk_refs.push_back(ch); pool.retain(std::vector<int>{ch}); }
        } else if ((int)build_reps.size() < kJitBatchMax && entry_offset + (int)build_reps.size() < kJitCycleEntries && index < kJitCycleBuilds)
          build_reps.push_back(r);                   // what does not fit this cycle is reported again by a later fill
      }
      if (!hit_reps.empty()) {
        xg_status_t st = jit_publish_from_host(g, hit_reps, hit_entries, stream);
        if (st != XG_OK) return st;
        for (size_t k = 0; k < hit_reps.size(); ++k) jit_record(g, std::vector<int32_t>{hit_reps[k]}, &hit_entries[k], &hit_counts[k], -1);
        j.n_pool_hits += (int)hit_reps.size();
      }
      if (!build_reps.empty()) {
        xg_status_t st = jit_enqueue_build(jp, g, build_reps, false, 0, entry_offset, index, stream);
        if (st != XG_OK) return st;
        entry_offset += (int)build_reps.size();
        ++index;
      }
    }
    if (!jp->flights.empty()) {
      XG_CUDA(cudaEventRecord(jp->ev, stream));
      jp->phase = 2;
      if (!wait) return XG_OK;
    }
  }
  return set_error(XG_ERR_TIMEOUT, "just-in-time service did not settle");
}

xg_status_t xg_compile_grammar(const xg_tokenizer_t* tok, xg_cache_pool_t* pool, xg_grammar_kind_t kind, const char* text, size_t len,
                               const char* root_rule, const xg_compile_options_t* opt, void* stream, xg_grammar_t** out) {
  NvtxRange nvtx_range("xg_compile_grammar");
  if (!out) return set_error(XG_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (!text) return set_error(XG_ERR_INVALID_ARG, "text is NULL");
  FrontendOptions fo;
  bool build_cache = tok != nullptr, compress = true, jit = false, count_visits = false;
  int jit_precompute = 0, repeat_threshold = 0, repeat_depth = 0;
  long long jit_arena_words = 0;
  if (opt) {
    if (opt->struct_size < 8) return set_error(XG_ERR_INVALID_ARG, "bad options struct_size");
    if (opt->inline_max_states >= 0) fo.inline_max_states = opt->inline_max_states;
    if (opt->struct_size >= 12 && opt->max_rule_states > 0) fo.max_rule_states = opt->max_rule_states;
    if (opt->struct_size >= 16 && opt->build_cache == 0) build_cache = false;
    if (opt->struct_size >= 20 && opt->no_state_compression != 0) compress = false;
    if (opt->struct_size >= 28 && opt->jit != 0) { jit = true; jit_precompute = std::max(0, opt->jit_precompute); }
    if (opt->struct_size >= 40 && opt->jit_arena_bytes > 0) jit_arena_words = std::max<long long>(1024, opt->jit_arena_bytes / 4);
    if (opt->struct_size >= 44 && opt->count_node_visits != 0) count_visits = true;
    if (opt->struct_size >= 48) repeat_threshold = opt->repeat_threshold;
    if (opt->struct_size >= 52 && opt->repeat_depth > 0) repeat_depth = opt->repeat_depth;
  }
  // counted repetitions (Section 3.6): on by default wherever the longest token is known
  if (tok && tok->dev.max_len > 0) repeat_depth = tok->dev.max_len;
  if (repeat_threshold == 0) repeat_threshold = kDefaultRepeatThreshold;
  if (repeat_threshold > 0 && repeat_depth > 0) { fo.repeat_threshold = repeat_threshold; fo.repeat_depth = repeat_depth; }
  if (pool && pool->impl->owner() != (const void*)tok) return set_error(XG_ERR_INVALID_ARG, "the pool belongs to another tokenizer");
  std::unique_ptr<xg_grammar> g(new xg_grammar());
  g->count_visits = count_visits;
  const double t0 = now_ms();
  try {
    FlatGrammar made = compile_frontend((int)kind, std::string(text, len), root_rule ? root_rule : "root", fo);
    if (made.rule_rep_lo.empty()) g->flat = std::move(made);
    else { g->flat = expand_counted_rules(made); g->base = std::move(made); g->counted = true; }
  } catch (const FrontendError& e) {
    return set_error(e.status, e.message);
  } catch (const std::bad_alloc&) {
    return set_error(XG_ERR_OOM, "out of host memory in the grammar front end");
  } catch (const std::exception& e) {
    return set_error(XG_ERR_PARSE, e.what());
  }
  const FlatGrammar& f = g->flat;
  g->stats.frontend_ms = now_ms() - t0;
  g->stats.n_rules = f.n_rules; g->stats.n_states = g->tables().n_states; g->stats.n_classes = f.n_classes;
  std::vector<int32_t> scannable;
  for (int s = 0; s < f.n_states; ++s) if (f.cedge_begin[s + 1] > f.cedge_begin[s]) scannable.push_back(s);
  g->stats.n_scannable = (int)scannable.size();
  if (!build_cache) { *out = g.release(); return XG_OK; }

  g->tok = tok;
  g->pool = pool ? pool->impl : std::make_shared<CachePool>((const void*)tok);
  g->entries.assign(f.n_states, EntryDev{});
  g->entry_counts.assign(f.n_states, make_int2(0, 0));
  g->entry_chunk.assign(f.n_states, -1);
  const std::shared_ptr<CachePool> pool_keep = g->pool;      // outlives the lock below on every path
  // what needs neither the pool nor the device comes before the lock, so that threads compiling side by side
  // only take turns for the pool lookups and the cache build: rule hashes and canonical orders (Section 3.3), and
  // the classes of states that share a cache entry (repetition state compression, Section 3.6)
  std::shared_ptr<const void> prepared;
  std::vector<int32_t> rep(f.n_states);
  const double t_pre = now_ms();
  try {
    prepared = prepare_interning(f);
    // (the classes only pay where a repetition of some length was expanded: inside a{0,16} they save a dozen entries
    // and cost as much host time as hashing the grammar)
    if (compress && tok->dev.max_len > 0 && f.max_expanded_repeat >= kShareEntriesFromRepeat) rep = bounded_equivalence(f, tok->dev.max_len);
    else for (int s = 0; s < f.n_states; ++s) rep[s] = s;
  } catch (const std::exception& e) {
    return set_error(XG_ERR_OOM, e.what());
  }
  const double pre_ms = now_ms() - t_pre;
  std::lock_guard<std::mutex> pool_lock(pool_keep->mu);
  const double t1 = now_ms();                                 // the cache build proper: not the wait for another thread's compile
  bool retained = false;
  auto fail = [&](xg_status_t status) {                       // the lock is held: give everything back without taking it again
    cudaDeviceSynchronize();
    if (retained) pool_keep->release_held(g->chunk_refs);
    g->chunk_refs.clear();
    pool_keep->free_plain(g->blob); pool_keep->free_plain(g->lookahead_arena);
    g->blob = g->lookahead_arena = nullptr;
    jit_release(g.get());
    xg_grammar_destroy(g.release());
    return status;
  };
  xg_status_t st = XG_OK;
  if (jit) {
    st = jit_allocate(g.get(), jit_arena_words);
    if (st != XG_OK) return fail(st);
  }
  st = upload_grammar(g.get(), (cudaStream_t)stream);
  if (st != XG_OK) return fail(st);
  // cross-grammar cache (Section 3.3): rules whose canonical structure is already in the pool
  // reuse its entries; the others are classified now and registered afterwards
  RuleInterning in;
  try {
    in = g->pool->intern(f, prepared);
  } catch (const std::exception& e) {
    return fail(set_error(XG_ERR_OOM, e.what()));
  }
  std::vector<int> rule_first(f.n_rules + 1, f.n_states);
  for (int s = f.n_states - 1; s >= 0; --s) rule_first[f.state_rule[s]] = s;
  std::vector<int> canon_of(f.n_states, -1);          // state -> canonical index inside its rule
  for (int r = 0; r < f.n_rules; ++r)
    for (size_t k = 0; k < in.canon[r].size(); ++k) canon_of[rule_first[r] + in.canon[r][k]] = (int)k;
  // (`rep`: states of a rule that no token of this vocabulary can tell apart share the entry of their class
  // representative)
  std::map<int, int> builder_of;                      // pool rule -> the rule of this grammar that builds it
  std::vector<int32_t> to_build;
  auto in_pool = [&](int s) {
    const PoolRule& pr = g->pool->rule(in.pool_id[f.state_rule[s]]);
    return pr.built && canon_of[s] < (int)pr.have.size() && pr.have[canon_of[s]];
  };
  for (int s : scannable) {
    const int r = f.state_rule[s];
    PoolRule& pr = g->pool->rule(in.pool_id[r]);
    if (in_pool(s)) {
      g->entries[s] = pr.entries[canon_of[s]];
      g->entry_counts[s] = pr.counts[canon_of[s]];
      ++g->stats.n_entries_reused;
      for (int c : pr.chunks) if (std::find(g->chunk_refs.begin(), g->chunk_refs.end(), c) == g->chunk_refs.end()) g->chunk_refs.push_back(c);
    } else {
      g->entries[s].kind = kEntryNotBuilt;
      auto it = builder_of.find(in.pool_id[r]);
      if (it == builder_of.end()) it = builder_of.emplace(in.pool_id[r], r).first;
      if (it->second == r) {
        if (rep[s] == s) to_build.push_back(s); else ++g->stats.n_entries_shared;
      }
    }
  }
  if (jit) {
    // configurable JIT (Section 3.5): only the K costliest of the missing entries are built now.
    // Cost of an entry = the tokens that pass its state's own first-byte test (the others are
    // rejected before a walk starts).
    std::vector<std::pair<int64_t, int32_t>> cost;
    for (int s : to_build) {
      int64_t c = 0;
      uint32_t own[8] = {};
      for (int e = f.cedge_begin[s]; e < f.cedge_begin[s + 1]; ++e)
        for (int w = 0; w < 8; ++w) own[w] |= f.class_bits[(size_t)f.cedge_class[e] * 8 + w];
      for (int b = 0; b < 256; ++b) if ((own[b >> 5] >> (b & 31)) & 1u) c += tok->first_byte_count[b];
      cost.emplace_back(-c, s);
    }
    std::sort(cost.begin(), cost.end());
    to_build.clear();
    for (int k = 0; k < (int)cost.size() && k < jit_precompute; ++k) to_build.push_back(cost[k].second);
    std::sort(to_build.begin(), to_build.end());
  }
  st = build_entries(g.get(), to_build, (cudaStream_t)stream);
  if (st != XG_OK) return fail(st);
  for (int s : scannable) {                           // the other members of each class
    if (rep[s] == s || g->entries[s].kind != kEntryNotBuilt) continue;
    auto it = builder_of.find(in.pool_id[f.state_rule[s]]);
    if (it == builder_of.end() || it->second != f.state_rule[s]) continue;
    g->entries[s] = g->entries[rep[s]]; g->entry_counts[s] = g->entry_counts[rep[s]]; g->entry_chunk[s] = g->entry_chunk[rep[s]];
  }
  for (auto& kv : builder_of) {
    PoolRule& pr = g->pool->rule(kv.first);
    const int r = kv.second;
    const int n_local = (int)in.canon[r].size();
    pr.entries.resize(n_local);
    pr.counts.resize(n_local);
    pr.have.resize(n_local, 0);
    for (int k = 0; k < n_local; ++k) {
      const int s = rule_first[r] + in.canon[r][k];
      if (pr.have[k] || g->entries[s].kind == kEntryNotBuilt) continue;
      pr.entries[k] = g->entries[s]; pr.counts[k] = g->entry_counts[s];
      pr.have[k] = 1;
      pr.built = true;
      const int c = g->entry_chunk[s];
      if (c >= 0 && std::find(pr.chunks.begin(), pr.chunks.end(), c) == pr.chunks.end()) { pr.chunks.push_back(c); g->pool->note_rule_in_chunk(kv.first, c); }
    }
    for (int c : pr.chunks) if (std::find(g->chunk_refs.begin(), g->chunk_refs.end(), c) == g->chunk_refs.end()) g->chunk_refs.push_back(c);
  }
  g->pool->retain(g->chunk_refs);
  retained = true;
  g->pool->enforce_limit();
  for (int s : scannable) {                           // duplicates of a rule inside this grammar
    const int r = f.state_rule[s];
    auto it = builder_of.find(in.pool_id[r]);
    if (it == builder_of.end() || it->second == r) continue;
    if (!in_pool(s)) continue;                        // a just-in-time grammar: not built yet
    const PoolRule& pr = g->pool->rule(in.pool_id[r]);
    g->entries[s] = pr.entries[canon_of[s]];
    g->entry_counts[s] = pr.counts[canon_of[s]];
    ++g->stats.n_entries_reused;
  }
  if (jit) {
    JitState& j = g->jit;
    j.rep = rep;
    j.in = in; j.canon_of = canon_of; j.rule_first = rule_first;
    j.status.assign(f.n_states, 2);
    std::vector<int32_t> count(f.n_states + 1, 0);
    for (int s2 = 0; s2 < f.n_states; ++s2) ++count[rep[s2] + 1];
    for (int s2 = 0; s2 < f.n_states; ++s2) count[s2 + 1] += count[s2];
    j.member_begin = count;
    j.members.resize(f.n_states);
    { std::vector<int32_t> at(count.begin(), count.end() - 1); for (int s2 = 0; s2 < f.n_states; ++s2) j.members[at[rep[s2]]++] = s2; }
    for (int s2 : scannable) if (rep[s2] == s2 && g->entries[s2].kind == kEntryNotBuilt) { j.status[s2] = 0; ++j.n_missing; }
    if (cudaMemcpy(j.d_rep, rep.data(), (size_t)f.n_states * 4, cudaMemcpyHostToDevice) != cudaSuccess)
      return fail(set_error(XG_ERR_CUDA, "upload of the state classes failed"));
    j.enabled = true;
  }
  st = upload_entry_headers(g.get(), (cudaStream_t)stream);       // now with the entry headers
  bool narrowed = false;
  if (st == XG_OK) st = narrow_check_lists(g.get(), scannable, rep, (cudaStream_t)stream, &narrowed);      // (synchronises after its first kernel)
  if (st == XG_OK && narrowed) st = upload_entry_headers(g.get(), (cudaStream_t)stream);       // and with this grammar's narrowed check lists
  if (st == XG_OK && cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) st = set_error(XG_ERR_CUDA, "cache build failed on the device");
  if (st != XG_OK) return fail(st);
  g->stats.cache_build_ms = now_ms() - t1 + pre_ms;
  g->stats.n_entries_built = (int)to_build.size();
  g->stats.pairs_classified = (int64_t)to_build.size() * tok->vocab_size;
  for (int s : scannable) {
    const EntryDev& e = g->entries[s];
    if (e.kind == kEntryNotBuilt) continue;
    const int2 c = g->entry_counts[s];
    g->stats.total_accepted += c.x;
    g->stats.total_uncertain += c.y;
    g->stats.total_checked += e.n_chk;
    g->max_check = std::max(g->max_check, (int)e.n_chk);
    g->stats.total_rejected += tok->vocab_size - c.x - c.y;
    g->stats.kind_count[e.kind]++;
    if (rep[s] == s) g->stats.cache_bytes += 4LL * ((e.kind == 2 ? tok->n_words : e.n_list) + 4LL * e.n_unc);
  }
  *out = g.release();
  return XG_OK;
}

xg_status_t xg_jit_service(xg_grammar_t* const* grammars, int32_t n, void* stream, int32_t wait, xg_jit_stats_t* out) {
  NvtxRange nvtx_range("xg_jit_service");
  if (n < 0 || (n > 0 && !grammars)) return set_error(XG_ERR_INVALID_ARG, "bad grammar array");
  std::vector<std::pair<CachePool*, std::vector<xg_grammar*>>> pools;      // the just-in-time grammars by pool
  for (int i = 0; i < n; ++i) {
    xg_grammar* g = grammars[i];
    if (!g) return set_error(XG_ERR_INVALID_ARG, "NULL grammar");
    if (!g->jit.enabled) continue;
    size_t k = 0;
    while (k < pools.size() && pools[k].first != g->pool.get()) ++k;
    if (k == pools.size()) pools.emplace_back(g->pool.get(), std::vector<xg_grammar*>());
    if (std::find(pools[k].second.begin(), pools[k].second.end(), g) == pools[k].second.end()) pools[k].second.push_back(g);
  }
  xg_jit_stats_t total{};
  for (auto& pg : pools) {
    std::lock_guard<std::mutex> lock(pg.first->mu);
    bool idle = false;
    xg_status_t st = jit_advance(*pg.first, pg.second, (cudaStream_t)stream, wait != 0, &idle);
    if (st != XG_OK) return st;
    for (xg_grammar* g : pg.second) {
      total.n_built += g->jit.n_built; total.n_pool_hits += g->jit.n_pool_hits;
      total.n_in_flight += g->jit.n_in_flight; total.n_missing += g->jit.n_missing;
    }
  }
  if (out) *out = total;
  return XG_OK;
}

void xg_grammar_destroy(xg_grammar_t* g) {
  if (!g) return;
  if (g->jit.d_rep || g->jit.slot >= 0) {
    std::lock_guard<std::mutex> lock(g->pool->mu);
    jit_release(g);
  }
  if (g->pool && (g->blob || g->lookahead_arena || !g->chunk_refs.empty())) {
    cudaDeviceSynchronize();             // its tables go back to the pool's slabs: nothing may still read them
    std::lock_guard<std::mutex> lock(g->pool->mu);
    g->pool->free_plain(g->blob);
    g->pool->free_plain(g->lookahead_arena);
    g->pool->release_held(g->chunk_refs);
  }
  delete g;
}

xg_status_t xg_grammar_get_tables(const xg_grammar_t* g, xg_grammar_tables_t* t) {
  if (!g || !t) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  const FlatGrammar& f = g->tables();
  t->rule_rep_lo = f.rule_rep_lo.empty() ? nullptr : f.rule_rep_lo.data();
  t->rule_rep_hi = f.rule_rep_hi.empty() ? nullptr : f.rule_rep_hi.data();
  t->cedge_iter = f.cedge_iter.empty() ? nullptr : f.cedge_iter.data();
  t->redge_iter = f.redge_iter.empty() ? nullptr : f.redge_iter.data();
  t->n_records = g->flat.n_states;
  t->n_rules = f.n_rules; t->n_states = f.n_states; t->n_classes = f.n_classes;
  t->n_class_edges = (int32_t)f.cedge_class.size(); t->n_ref_edges = (int32_t)f.redge_rule.size();
  t->root_rule = f.root_rule; t->root_nullable = f.root_nullable;
  t->rule_start = f.rule_start.data(); t->state_rule = f.state_rule.data(); t->state_final = f.state_final.data();
  t->cedge_begin = f.cedge_begin.data(); t->cedge_class = f.cedge_class.data(); t->cedge_target = f.cedge_target.data();
  t->redge_begin = f.redge_begin.data(); t->redge_rule = f.redge_rule.data(); t->redge_target = f.redge_target.data();
  t->class_bits = f.class_bits.data();
  return XG_OK;
}

xg_status_t xg_grammar_record_of(const xg_grammar_t* g, int32_t state, int32_t count, int32_t* record) {
  if (!g || !record) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  const FlatGrammar& f = g->tables();
  if (state < 0 || state >= f.n_states || count < 0) return set_error(XG_ERR_INVALID_ARG, "state or count out of range");
  if (!g->counted || state < g->flat.rep_first) { *record = state; return XG_OK; }
  if (count >= f.rule_rep_hi[f.state_rule[state]]) return set_error(XG_ERR_INVALID_ARG, "count beyond the repetition's upper bound");
  *record = record_of(g->flat, state, count);
  return XG_OK;
}

xg_status_t xg_grammar_get_rule_hashes(const xg_grammar_t* g, uint64_t* out) {
  if (!g || !out) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  try {
    RuleInterning in = structural_hashes(g->flat);
    for (int r = 0; r < g->flat.n_rules; ++r) out[r] = in.hash[r];
  } catch (const std::exception& e) {
    return set_error(XG_ERR_OOM, e.what());
  }
  return XG_OK;
}

xg_status_t xg_grammar_get_state_classes(const xg_grammar_t* g, int32_t depth, int32_t* out) {
  if (!g || !out) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  if (g->counted) return set_error(XG_ERR_UNSUPPORTED, "the grammar has counted repetitions: its records are the classes");
  if (depth < 0) {
    if (!g->tok) return set_error(XG_ERR_INVALID_ARG, "depth < 0 needs a grammar compiled with a tokenizer");
    depth = g->tok->dev.max_len;
  }
  try {
    const std::vector<int32_t> rep = bounded_equivalence(g->flat, depth);
    std::memcpy(out, rep.data(), rep.size() * sizeof(int32_t));
  } catch (const std::bad_alloc&) {
    return set_error(XG_ERR_OOM, "out of host memory");
  }
  return XG_OK;
}

xg_status_t xg_grammar_get_cache_entry(const xg_grammar_t* g, int32_t state, xg_cache_entry_view_t* view) {
  if (!g || !view) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  if (!g->tok) return set_error(XG_ERR_INVALID_ARG, "the grammar was compiled without a cache");
  const FlatGrammar& f = g->flat;
  if (state < 0 || state >= f.n_states || f.cedge_begin[state + 1] == f.cedge_begin[state]) return set_error(XG_ERR_INVALID_ARG, "state is not scannable");
  const EntryDev& e = g->entries[state];
  if (e.kind == kEntryNotBuilt) return set_error(XG_ERR_INVALID_ARG, "the entry of this state has not been built yet (just-in-time grammar)");
  const int2 c = g->entry_counts[state];
  XG_CUDA(cudaDeviceSynchronize());
  view->state = state; view->kind = e.kind;
  view->n_accepted = c.x; view->n_uncertain = c.y; view->n_rejected = g->tok->vocab_size - c.x - c.y;
  view->n_list = e.n_list; view->list = nullptr; view->bitset = nullptr;
  if (e.kind == XG_STORE_BITSET) {
    g->view_bits.resize(g->tok->n_words);
    XG_CUDA(cudaMemcpy(g->view_bits.data(), e.data, g->view_bits.size() * 4, cudaMemcpyDeviceToHost));
    view->bitset = g->view_bits.data();
  } else {
    g->view_list.resize(std::max(e.n_list, 1));
    if (e.n_list) XG_CUDA(cudaMemcpy(g->view_list.data(), e.data, (size_t)e.n_list * 4, cudaMemcpyDeviceToHost));
    view->list = g->view_list.data();
  }
  g->view_unc.resize(std::max(e.n_unc, 1));
  if (e.n_unc) XG_CUDA(cudaMemcpy(g->view_unc.data(), e.unc_id, (size_t)e.n_unc * 4, cudaMemcpyDeviceToHost));
  view->uncertain = g->view_unc.data();
  return XG_OK;
}

xg_status_t xg_grammar_stats(const xg_grammar_t* g, xg_grammar_stats_t* out) {
  if (!g || !out) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  *out = g->stats;
  return XG_OK;
}

// ---------------------------------------------------------------------------------------------
// matchers
// ---------------------------------------------------------------------------------------------
xg_status_t xg_matcher_create(const xg_grammar_t* g, const xg_matcher_options_t* opt, void* stream, xg_matcher_t** out) {
  if (!out) return set_error(XG_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (!g || !g->tok || !g->dev) return set_error(XG_ERR_INVALID_ARG, "the grammar has no compiled cache");
  int max_sets = 16384, max_items = 0;
  if (opt) {
    if (opt->struct_size >= 8 && opt->max_sets > 0) max_sets = opt->max_sets;
    if (opt->struct_size >= 12 && opt->max_items > 0) max_items = opt->max_items;
  }
  if (max_sets < 2) return set_error(XG_ERR_INVALID_ARG, "max_sets must be at least 2");
  if (max_items <= 0) max_items = 4 * max_sets;
  std::unique_ptr<xg_matcher> m(new xg_matcher());
  m->grammar = g;
  const size_t o_plan = 256, o_items = o_plan + ((sizeof(StepPlan) + 255) & ~size_t(255)), o_org = o_items + (size_t)max_items * 4,
               o_sb = o_org + (size_t)max_items * 4;
  const size_t o_slow_st = (o_sb + ((size_t)max_sets + 1) * 4 + 255) & ~size_t(255), o_slow_org = o_slow_st + (size_t)kSlowCap * 4,
               o_slow_lsb = o_slow_org + (size_t)kSlowCap * 4, o_slow_q = o_slow_lsb + (size_t)(kSlowMaxBytes + 2) * 4;
  const size_t total = o_slow_q + (size_t)kSlowQueue * 4;
  XG_CUDA(cudaMalloc(&m->block, total));
  uint8_t* d = (uint8_t*)m->block;
  MatcherDev h{};
  h.grammar = g->dev;
  h.item_state = (uint32_t*)(d + o_items);
  h.item_origin = (int32_t*)(d + o_org);
  h.set_begin = (int32_t*)(d + o_sb);
  h.cap_sets = max_sets; h.cap_items = max_items;
  h.plan = (StepPlan*)(d + o_plan);
  h.slow_st = (uint32_t*)(d + o_slow_st); h.slow_org = (int32_t*)(d + o_slow_org);
  h.slow_lsb = (int32_t*)(d + o_slow_lsb); h.slow_q = (int32_t*)(d + o_slow_q);
  m->dev = (MatcherDev*)d;
  cudaError_t err = cudaMemcpyAsync(m->dev, &h, sizeof h, cudaMemcpyHostToDevice, (cudaStream_t)stream);
  if (err == cudaSuccess) { matcher_reset_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(m->dev); err = cudaGetLastError(); }
  if (err == cudaSuccess) err = cudaStreamSynchronize((cudaStream_t)stream);     // `h` is a stack object
  if (err != cudaSuccess) { cudaFree(m->block); return set_error(XG_ERR_CUDA, std::string("matcher init: ") + cudaGetErrorString(err)); }
  *out = m.release();
  return XG_OK;
}

xg_status_t xg_matcher_reset(xg_matcher_t* m, void* stream) {
  if (!m) return set_error(XG_ERR_INVALID_ARG, "NULL matcher");
  matcher_reset_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(m->dev);
  XG_CUDA(cudaGetLastError());
  return XG_OK;
}

void xg_matcher_destroy(xg_matcher_t* m) {
  if (!m) return;
  if (m->grammar && m->grammar->tok) {       // forget cached batches that contain this matcher
    const xg_tokenizer* t = m->grammar->tok;
    std::lock_guard<std::mutex> lock(t->mu);
    for (auto& s : t->batches.slots)
      if (std::find(s.key.begin(), s.key.end(), m) != s.key.end()) s.key.clear();
  }
  cudaFree(m->block);
  delete m;
}

xg_status_t xg_matcher_is_terminated(const xg_matcher_t* m, void* stream, int32_t* out) {
  if (!m || !out) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  MatcherDev h;
  XG_CUDA(cudaMemcpyAsync(&h, m->dev, sizeof h, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  XG_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  *out = h.terminated ? 1 : 0;
  return XG_OK;
}

xg_status_t xg_matcher_next_fill_work(const xg_matcher_t* m, void* stream, xg_fill_work_t* out) {
  if (!m || !out) return set_error(XG_ERR_INVALID_ARG, "NULL argument");
  const xg_grammar* g = m->grammar;
  MatcherDev h;
  XG_CUDA(cudaMemcpyAsync(&h, m->dev, sizeof h, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  XG_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  std::unique_ptr<StepPlan> plan(new StepPlan());
  XG_CUDA(cudaMemcpyAsync(plan.get(), h.plan, sizeof(StepPlan), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  XG_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  xg_fill_work_t w{};
  const int64_t W = g->tok->n_words;
  w.row_bytes = 4 * W;
  if (!h.terminated && !plan->overflow) {
    w.n_merge = plan->n_merge; w.n_check = plan->n_check; w.n_missing = plan->n_missing;
    for (int k = 0; k < plan->n_merge; ++k) {
      const EntryDev& e = g->entries[plan->merge_state[k]];
      if (e.kind == XG_STORE_BITSET) w.merge_bytes += 4 * W;
      else if (e.kind == XG_STORE_ACCEPT_LIST) w.merge_bytes += 4LL * e.n_list;
      else if (e.kind == XG_STORE_REJECT_LIST) w.merge_bytes += 4LL * e.n_list + 4LL * e.n_unc;
    }
    w.check_tokens = plan->n_check ? plan->check_cum[plan->n_check] : 0;
    w.check_bytes = 12 * w.check_tokens;
  }
  *out = w;
  return XG_OK;
}

// (re)allocate the batch tables for `cap` requests per composition; only when a batch is larger than any before
static xg_status_t grow_batch_tables(BatchTables& bt, int cap) {
  XG_CUDA(cudaDeviceSynchronize());              // the old tables may still be in use
  for (auto& s : bt.slots) if (s.uploaded) cudaEventDestroy(s.uploaded);
  bt.slots.clear();
  cudaFree(bt.dev_slab); cudaFree(bt.words);
  if (bt.host_slab) cudaFreeHost(bt.host_slab);
  bt.dev_slab = nullptr; bt.words = nullptr; bt.host_slab = nullptr; bt.cap = 0;
  XG_CUDA(cudaMalloc(&bt.dev_slab, sizeof(void*) * (size_t)cap * kBatchEntries));
  XG_CUDA(cudaMalloc(&bt.words, sizeof(int32_t) * 2 * (size_t)cap));
  XG_CUDA(cudaHostAlloc(&bt.host_slab, sizeof(void*) * (size_t)cap * kBatchEntries, cudaHostAllocDefault));
  bt.cap = cap;
  bt.slots.resize(kBatchEntries);
  for (int k = 0; k < kBatchEntries; ++k) {
    BatchSlot& s = bt.slots[k];
    s.dev_matchers = bt.dev_slab + (size_t)k * cap;
    s.staging = bt.host_slab + (size_t)k * cap;
    s.status = bt.words; s.done_count = bt.words + cap;
    XG_CUDA(cudaEventCreateWithFlags(&s.uploaded, cudaEventDisableTiming));
  }
  return XG_OK;
}

// device-side array of matcher pointers for this batch composition (see BatchTables)
static xg_status_t batch_slot(xg_matcher_t* const* matchers, int32_t batch, cudaStream_t stream, const xg_tokenizer** tok_out, BatchSlot** slot_out) {
  if (!matchers || batch <= 0) return set_error(XG_ERR_INVALID_ARG, "empty batch");
  if (batch > 65535) return set_error(XG_ERR_INVALID_ARG, "batch larger than 65535");
  for (int i = 0; i < batch; ++i) if (!matchers[i]) return set_error(XG_ERR_INVALID_ARG, "NULL matcher in batch");
  const xg_tokenizer* tok = matchers[0]->grammar->tok;
  for (int i = 1; i < batch; ++i) if (matchers[i]->grammar->tok != tok) return set_error(XG_ERR_INVALID_ARG, "matchers of one batch must share a tokenizer");
  std::lock_guard<std::mutex> lock(tok->mu);
  BatchTables& bt = tok->batches;
  if (batch > bt.cap) {
    int cap = std::max(256, bt.cap);
    while (cap < batch) cap *= 2;
    xg_status_t st = grow_batch_tables(bt, cap);
    if (st != XG_OK) return st;
  }
  BatchSlot* hit = nullptr;
  for (auto& s : bt.slots)
    if ((int)s.key.size() == batch && std::memcmp(s.key.data(), matchers, sizeof(void*) * batch) == 0) { hit = &s; break; }
  if (!hit) {
    BatchSlot* victim = nullptr;
    for (auto& s : bt.slots) {
      if (s.in_graph && !s.key.empty()) continue;
      if (s.key.empty()) { victim = &s; break; }
      if (!victim || s.last_use < victim->last_use) victim = &s;
    }
    if (!victim) return set_error(XG_ERR_CAPACITY, "every cached batch composition belongs to a captured graph");
    if (victim->upload_recorded) XG_CUDA(cudaEventSynchronize(victim->uploaded));      // its staging buffer is free again (long done, normally)
    for (int i = 0; i < batch; ++i) victim->staging[i] = matchers[i]->dev;
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    XG_CUDA(cudaStreamIsCapturing(stream, &capturing));
    XG_CUDA(cudaMemcpyAsync(victim->dev_matchers, victim->staging, sizeof(void*) * batch, cudaMemcpyHostToDevice, stream));
    victim->in_graph = capturing != cudaStreamCaptureStatusNone;
    victim->upload_recorded = false;
    if (!victim->in_graph) { XG_CUDA(cudaEventRecord(victim->uploaded, stream)); victim->upload_recorded = true; }
    victim->key.assign(matchers, matchers + batch);
    hit = victim;
  }
  hit->last_use = ++tok->use_counter;
  *tok_out = tok;
  *slot_out = hit;
  return XG_OK;
}

// Does a grammar of the batch have counted repetitions (Section 3.6)?  Then the step kernels decode the count out of
// every state word; otherwise the variants without that decode run.
static bool batch_has_counted_rules(xg_matcher_t* const* matchers, int32_t batch) {
  for (int i = 0; i < batch; ++i) if (matchers[i]->grammar->counted) return true;
  return false;
}

static xg_status_t apply_rows(void* logits_dev, xg_dtype_t dtype, int32_t rows, int32_t vocab_size, int64_t logits_row_stride_elems,
                              const int32_t* bitmask_dev, int64_t mask_row_stride_words, const int32_t* row_indices_dev, void* stream);

// accept (when token_ids_dev is given), fill, and apply (when logits_dev is given)
static xg_status_t accept_and_fill(xg_matcher_t* const* matchers, int32_t batch, const int32_t* token_ids_dev, int32_t* accept_status_dev,
                                   int restart_on_eos, int32_t* bitmask_dev, int64_t row_stride_words, int32_t* status_dev, void* stream,
                                   void* logits_dev = nullptr, xg_dtype_t dtype = XG_F32, int64_t logits_row_stride_elems = 0) {
  const xg_tokenizer* tok = nullptr;
  BatchSlot* slot = nullptr;
  xg_status_t st = batch_slot(matchers, batch, (cudaStream_t)stream, &tok, &slot);
  if (st != XG_OK) return st;
  if (!bitmask_dev || row_stride_words < tok->n_words) return set_error(XG_ERR_INVALID_ARG, "bad bitmask buffer");
  const int W = tok->n_words;
  if ((W + kMaxClusterBlocks - 1) / kMaxClusterBlocks <= kMergeMaxChunkWords) {
    // One launch: a cluster of blocks per request keeps the row in distributed shared memory.
    // Eight blocks per request; 256 threads each while that leaves the whole batch resident (the
    // kernel runs at 64 registers per thread: 1024 threads per SM), else 128.
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int per_request = sms * 1024 / batch;
    int blocks = kMaxClusterBlocks, threads = 256;
    if (per_request < 2048) threads = 128;     // measured: narrower blocks than this are slower even at batch 256
    // more requests than fit the SMs at eight blocks each (8 blocks of 128 threads per SM): clusters of four, so that
    // the launch is still one wave (C5, batch 256: fill 74 -> 69 us)
    if (batch * blocks > sms * 8 && (W + 3) / 4 <= kMergeMaxChunkWords) blocks = 4;
    const size_t smem = 2 * sizeof(uint32_t) * (size_t)((W + blocks - 1) / blocks);
    MatcherDev* const* dm = slot->dev_matchers;
    // requests with hundreds of uncertain candidates are possible only where some entry has a long check list
    bool heavy = false;
    for (int i = 0; i < batch && !heavy; ++i) heavy = matchers[i]->grammar->max_check >= 1024;
    const dim3 grid(blocks, batch), block(threads);
    cudaStream_t cs = (cudaStream_t)stream;
    const long long stride_w = (long long)row_stride_words, stride_l = (long long)logits_row_stride_elems;
    const bool counts = batch_has_counted_rules(matchers, batch);
#define XG_FILL_C(ACCEPT, ELEMS, HEAVY, COUNTS, TOK, AST, RST, LOGITS)                                                                              \
    XG_CUDA(launch_step_kernel(fill_cluster_kernel<ACCEPT, ELEMS, HEAVY, COUNTS>, grid, block, smem, cs, blocks, dm, tok->dev, bitmask_dev, stride_w, \
                               status_dev, (const int32_t*)(TOK), (int32_t*)(AST), (int)(RST), (void*)(LOGITS), stride_l))
#define XG_FILL(ACCEPT, ELEMS, HEAVY, TOK, AST, RST, LOGITS) \
    do { if (counts) XG_FILL_C(ACCEPT, ELEMS, HEAVY, true, TOK, AST, RST, LOGITS); else XG_FILL_C(ACCEPT, ELEMS, HEAVY, false, TOK, AST, RST, LOGITS); } while (0)
    if (token_ids_dev) { if (heavy) XG_FILL(true, 0, true, token_ids_dev, accept_status_dev, restart_on_eos, nullptr); else XG_FILL(true, 0, false, token_ids_dev, accept_status_dev, restart_on_eos, nullptr); }
    else if (!logits_dev) { if (heavy) XG_FILL(false, 0, true, nullptr, nullptr, 0, nullptr); else XG_FILL(false, 0, false, nullptr, nullptr, 0, nullptr); }
    else if (dtype == XG_BF16) { if (heavy) XG_FILL(false, 8, true, nullptr, nullptr, 0, logits_dev); else XG_FILL(false, 8, false, nullptr, nullptr, 0, logits_dev); }
    else { if (heavy) XG_FILL(false, 4, true, nullptr, nullptr, 0, logits_dev); else XG_FILL(false, 4, false, nullptr, nullptr, 0, logits_dev); }
#undef XG_FILL
#undef XG_FILL_C
    return XG_OK;
  }
  if (token_ids_dev) {
    XG_CUDA(launch_step_kernel(batch_has_counted_rules(matchers, batch) ? accept_kernel<true> : accept_kernel<false>, dim3((batch + 3) / 4), dim3(128), 0,
                               (cudaStream_t)stream, 1, (MatcherDev* const*)slot->dev_matchers, (int)batch, tok->dev, token_ids_dev, accept_status_dev, restart_on_eos));
  }
  int chunks = std::max((W + kMergeMaxChunkWords - 1) / kMergeMaxChunkWords, std::min(8, (W + 127) / 128));
  dim3 grid_merge(chunks, batch);
  merge_kernel<<<grid_merge, 256, 0, (cudaStream_t)stream>>>(slot->dev_matchers, tok->dev, bitmask_dev, (long long)row_stride_words,
                                                             status_dev, slot->status, slot->done_count);
  dim3 grid_check(8, batch);
  check_kernel<<<grid_check, 256, 0, (cudaStream_t)stream>>>(slot->dev_matchers, tok->dev, bitmask_dev, (long long)row_stride_words,
                                                             status_dev, slot->status, slot->done_count);
  XG_CUDA(cudaGetLastError());
  if (logits_dev) return apply_rows(logits_dev, dtype, batch, tok->vocab_size, logits_row_stride_elems, bitmask_dev, row_stride_words, nullptr, stream);
  return XG_OK;
}

xg_status_t xg_fill_next_token_bitmask(xg_matcher_t* const* matchers, int32_t batch, int32_t* bitmask_dev, int64_t row_stride_words,
                                       int32_t* status_dev, void* stream) {
  NvtxRange nvtx_range("xg_fill_next_token_bitmask");
  return accept_and_fill(matchers, batch, nullptr, nullptr, 0, bitmask_dev, row_stride_words, status_dev, stream);
}

xg_status_t xg_accept_token_and_fill_next_bitmask(xg_matcher_t* const* matchers, int32_t batch, const int32_t* token_ids_dev,
                                                  int32_t* accept_status_dev, int32_t restart_on_eos, int32_t* bitmask_dev,
                                                  int64_t row_stride_words, int32_t* fill_status_dev, void* stream) {
  NvtxRange nvtx_range("xg_accept_token_and_fill_next_bitmask");
  if (!token_ids_dev) return set_error(XG_ERR_INVALID_ARG, "token_ids_dev is NULL");
  return accept_and_fill(matchers, batch, token_ids_dev, accept_status_dev, restart_on_eos ? 1 : 0, bitmask_dev, row_stride_words, fill_status_dev, stream);
}

xg_status_t xg_fill_and_apply_token_bitmask(xg_matcher_t* const* matchers, int32_t batch, int32_t* bitmask_dev, int64_t row_stride_words,
                                            int32_t* status_dev, void* logits_dev, xg_dtype_t dtype, int64_t logits_row_stride_elems,
                                            void* stream) {
  NvtxRange nvtx_range("xg_fill_and_apply_token_bitmask");
  if (!logits_dev) return set_error(XG_ERR_INVALID_ARG, "logits_dev is NULL");
  if (dtype != XG_F32 && dtype != XG_BF16) return set_error(XG_ERR_INVALID_ARG, "unknown dtype");
  if (!matchers || batch <= 0 || !matchers[0]) return set_error(XG_ERR_INVALID_ARG, "empty batch");
  const int elt = dtype == XG_BF16 ? 2 : 4;
  if (logits_row_stride_elems < matchers[0]->grammar->tok->vocab_size) return set_error(XG_ERR_INVALID_ARG, "bad shape or stride");
  if (((uintptr_t)logits_dev & 15) || ((logits_row_stride_elems * elt) & 15))
    return set_error(XG_ERR_INVALID_ARG, "logits rows must start on 16-byte boundaries");
  return accept_and_fill(matchers, batch, nullptr, nullptr, 0, bitmask_dev, row_stride_words, status_dev, stream, logits_dev, dtype, logits_row_stride_elems);
}

// ---------------------------------------------------------------------------------------------
// the per-step fill for callers that must not allocate: request table, status words and
// completion counters live in a fixed array inside the library image instead of cudaMalloc'ed
// per-batch buffers
// ---------------------------------------------------------------------------------------------
struct StaticFillScratch {
  MatcherDev* matchers[XG_STATIC_FILL_MAX_BATCH];
  int32_t status[XG_STATIC_FILL_MAX_BATCH];
  int32_t done_count[XG_STATIC_FILL_MAX_BATCH];
};
static __device__ __align__(256) unsigned char g_static_fill_scratch[sizeof(StaticFillScratch)];

// the request table of one call, passed to the set-up kernel by value (8 KiB of launch parameters)
struct StaticFillTable {
  MatcherDev* matchers[XG_STATIC_FILL_MAX_BATCH];
};
static __global__ void static_fill_setup_kernel(StaticFillScratch* sc, const __grid_constant__ StaticFillTable table, int batch) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= batch) return;
  sc->matchers[i] = table.matchers[i];
  sc->status[i] = 0;
  sc->done_count[i] = 0;
}

// The symbol above is only a host-side stand-in; kernels need its device address, which differs
// per device.  Looked up once per device, with that device current.
static xg_status_t static_fill_scratch(StaticFillScratch** out) {
  static std::mutex mu;
  static StaticFillScratch* by_device[64] = {};
  int dev = 0;
  XG_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return set_error(XG_ERR_UNSUPPORTED, "device ordinal above 63");
  std::lock_guard<std::mutex> lock(mu);
  if (!by_device[dev]) {
    void* p = nullptr;
    XG_CUDA(cudaGetSymbolAddress(&p, g_static_fill_scratch));
    by_device[dev] = (StaticFillScratch*)p;
  }
  *out = by_device[dev];
  return XG_OK;
}

xg_status_t xg_fill_next_token_bitmask_static(xg_matcher_t* const* matchers, int32_t batch, int32_t* bitmask_dev, int64_t row_stride_words,
                                              int32_t* status_dev, void* stream) {
  NvtxRange nvtx_range("xg_fill_next_token_bitmask_static");
  if (!matchers || batch <= 0) return set_error(XG_ERR_INVALID_ARG, "empty batch");
  if (batch > XG_STATIC_FILL_MAX_BATCH)
    return set_error(XG_ERR_CAPACITY, "batch of " + std::to_string(batch) + " requests exceeds the static scratch limit of " +
                                          std::to_string(XG_STATIC_FILL_MAX_BATCH) + "; use xg_fill_next_token_bitmask or split the batch");
  StaticFillTable table;
  for (int i = 0; i < batch; ++i) {
    if (!matchers[i]) return set_error(XG_ERR_INVALID_ARG, "NULL matcher in batch");
    if (matchers[i]->grammar->tok != matchers[0]->grammar->tok) return set_error(XG_ERR_INVALID_ARG, "matchers of one batch must share a tokenizer");
    table.matchers[i] = matchers[i]->dev;
  }
  const xg_tokenizer* tok = matchers[0]->grammar->tok;
  if (!bitmask_dev || row_stride_words < tok->n_words) return set_error(XG_ERR_INVALID_ARG, "bad bitmask buffer");
  StaticFillScratch* sc = nullptr;
  xg_status_t st = static_fill_scratch(&sc);
  if (st != XG_OK) return st;
  cudaStream_t cs = (cudaStream_t)stream;
  // the array keeps the previous call's contents: the request table is rewritten and the words cleared by a small
  // kernel that gets the table as a launch parameter (no host buffer has to outlive the call)
  static_fill_setup_kernel<<<(batch + 255) / 256, 256, 0, cs>>>(sc, table, batch);
  const int W = tok->n_words;
  int chunks = std::max((W + kMergeMaxChunkWords - 1) / kMergeMaxChunkWords, std::min(8, (W + 127) / 128));
  merge_kernel<<<dim3(chunks, batch), 256, 0, cs>>>(sc->matchers, tok->dev, bitmask_dev, (long long)row_stride_words, status_dev, sc->status, sc->done_count);
  check_kernel<<<dim3(8, batch), 256, 0, cs>>>(sc->matchers, tok->dev, bitmask_dev, (long long)row_stride_words, status_dev, sc->status, sc->done_count);
  XG_CUDA(cudaGetLastError());
  return XG_OK;
}

xg_status_t xg_accept_token(xg_matcher_t* const* matchers, int32_t batch, const int32_t* token_ids_dev, int32_t* status_dev, void* stream) {
  return xg_accept_token_ex(matchers, batch, token_ids_dev, status_dev, 0, stream);
}

xg_status_t xg_accept_token_ex(xg_matcher_t* const* matchers, int32_t batch, const int32_t* token_ids_dev, int32_t* status_dev,
                               int32_t restart_on_eos, void* stream) {
  NvtxRange nvtx_range("xg_accept_token");
  const xg_tokenizer* tok = nullptr;
  BatchSlot* slot = nullptr;
  xg_status_t st = batch_slot(matchers, batch, (cudaStream_t)stream, &tok, &slot);
  if (st != XG_OK) return st;
  if (!token_ids_dev) return set_error(XG_ERR_INVALID_ARG, "token_ids_dev is NULL");
  XG_CUDA(launch_step_kernel(batch_has_counted_rules(matchers, batch) ? accept_kernel<true> : accept_kernel<false>, dim3((batch + 3) / 4), dim3(128), 0,
                             (cudaStream_t)stream, 1, (MatcherDev* const*)slot->dev_matchers, (int)batch, tok->dev, token_ids_dev, status_dev, restart_on_eos ? 1 : 0));
  return XG_OK;
}

xg_status_t xg_apply_token_bitmask(void* logits_dev, xg_dtype_t dtype, int32_t batch, int32_t vocab_size, int64_t logits_row_stride_elems,
                                   const int32_t* bitmask_dev, int64_t mask_row_stride_words, const int32_t* row_indices_dev,
                                   int32_t n_rows, void* stream) {
  NvtxRange nvtx_range("xg_apply_token_bitmask");
  const int rows = row_indices_dev ? n_rows : batch;
  return apply_rows(logits_dev, dtype, rows, vocab_size, logits_row_stride_elems, bitmask_dev, mask_row_stride_words, row_indices_dev, stream);
}

static xg_status_t apply_rows(void* logits_dev, xg_dtype_t dtype, int32_t rows, int32_t vocab_size, int64_t logits_row_stride_elems,
                              const int32_t* bitmask_dev, int64_t mask_row_stride_words, const int32_t* row_indices_dev, void* stream) {
  if (!logits_dev || !bitmask_dev) return set_error(XG_ERR_INVALID_ARG, "NULL buffer");
  if (dtype != XG_F32 && dtype != XG_BF16) return set_error(XG_ERR_INVALID_ARG, "unknown dtype");
  if (vocab_size <= 0 || logits_row_stride_elems < vocab_size || mask_row_stride_words < (vocab_size + 31) / 32)
    return set_error(XG_ERR_INVALID_ARG, "bad shape or stride");
  if (rows == 0 && row_indices_dev) return XG_OK;
  if (rows <= 0) return set_error(XG_ERR_INVALID_ARG, "no rows");
  const int elt = dtype == XG_BF16 ? 2 : 4;
  if (((uintptr_t)logits_dev & 15) || ((logits_row_stride_elems * elt) & 15))
    return set_error(XG_ERR_INVALID_ARG, "logits rows must start on 16-byte boundaries");
  const int elems = 16 / elt;
  const int n_vec = vocab_size / elems;
  // Enough blocks per row that every thread makes one pass of four vectors (measured: C3 9.4 us per launch against
  // 11.1 with half as many blocks and two passes, C5 27.7 against 31.7; more and narrower passes are slower again),
  // and for small batches at least about eight blocks of 256 threads per SM in total.
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int per_row_max = std::max(1, (n_vec + 255) / 256);
  const int one_pass = (n_vec + 1023) / 1024;
  const int bx = std::max(1, std::min(per_row_max, std::max(one_pass, (sms * 8 + rows / 2) / rows)));
  if (rows > 65535) return set_error(XG_ERR_INVALID_ARG, "more than 65535 rows");
  dim3 grid(bx, rows);
  if (dtype == XG_BF16)
    XG_CUDA(launch_step_kernel(apply_kernel<8>, grid, dim3(256), 0, (cudaStream_t)stream, 1, logits_dev, (int)vocab_size, (long long)logits_row_stride_elems,
                               (const uint32_t*)bitmask_dev, (long long)mask_row_stride_words, row_indices_dev));
  else
    XG_CUDA(launch_step_kernel(apply_kernel<4>, grid, dim3(256), 0, (cudaStream_t)stream, 1, logits_dev, (int)vocab_size, (long long)logits_row_stride_elems,
                               (const uint32_t*)bitmask_dev, (long long)mask_row_stride_words, row_indices_dev));
  return XG_OK;
}

}  // extern "C"
