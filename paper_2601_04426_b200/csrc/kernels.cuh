// CUDA kernels of the token-mask path (sm_100a).  Integer / bit work only: nothing here is a
// dense contraction, so no tensor cores; the rules that matter are coalesced streaming, work
// that follows the trie order of the vocabulary, and grids sized to fill 148 SMs.
#pragma once
#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "device_types.h"

namespace xg {

enum : int { kWalkUncertain = 1, kWalkOverflow = 2 };

#ifdef XG_DEBUG_BOUNDS
// first violation: 1 << 63 | what << 48 | (index & 0xFFFFFF) << 24 | (limit & 0xFFFFFF)
__device__ unsigned long long g_bounds_violation = 0ull;
__device__ __forceinline__ bool bound_ok(long long index, long long limit, int what) {
  if (index >= 0 && index < limit) return true;
  atomicCAS(&g_bounds_violation, 0ull, (1ull << 63) | ((unsigned long long)what << 48) | (((unsigned long long)index & 0xFFFFFFull) << 24) | ((unsigned long long)limit & 0xFFFFFFull));
  return false;
}
#endif

// Programmatic dependent launch: the three kernels of a decode step are short, so the gap between
// one kernel's end and the next one's start is a large share of the step.  Each of them lets the
// next kernel of the stream be scheduled at once (its blocks become resident as room appears) and
// itself waits, before it touches any memory, until the previous kernel has finished and its
// writes are visible.  The order of all memory accesses is that of plain stream order.  Both are
// no-ops for a launch without the programmatic-serialisation attribute.
__device__ __forceinline__ void step_kernel_prologue() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

constexpr int kFastCap = 48;     // items a token walk may create before it falls back
constexpr int kFastMaxBytes = 32;
constexpr int kSlowCap = 2048;
constexpr int kSlowMaxBytes = 255;

// ------------------------------------------------------------------------------------------
// The token walk: Earley scan / complete over the bytes of one token (appendix "Earley's
// Parsing Algorithm"), on kernel items only.
//
// Chart: history sets 0..n given by (h_st, h_org, h_sb); an initial set (i_st, i_org, i_cnt)
// with chart index i_idx >= n (it may simply be history set n); the walk appends new sets to
// (st, org) with boundaries lsb[j] .. lsb[j+1] for the set reached after byte j (1-based), chart
// index i_idx + j.  Origin -1 stands for the unknown context of a cache entry (Section 3.4):
// completing such an item cannot advance anything known here; the byte offsets at which that
// happens (with bytes left) are the token's exits from its rule.
//
// Returns the number of bytes after which the set was still non-empty (len = token survives).
// ------------------------------------------------------------------------------------------
struct Chart {
  const uint32_t* h_st;
  const int32_t* h_org;
  const int32_t* h_sb;
  int n;
  const uint32_t* i_st;
  const int32_t* i_org;
  int i_cnt, i_idx;
  int h_items;          // items in the history (bounds-checking build)
};

__device__ __forceinline__ Chart chart_of_history(const uint32_t* h_st, const int32_t* h_org, const int32_t* h_sb, int n) {
  Chart c;
  c.h_st = h_st; c.h_org = h_org; c.h_sb = h_sb; c.n = n;
  const int b = h_sb[n];
  c.i_st = h_st + b; c.i_org = h_org + b; c.i_cnt = h_sb[n + 1] - b; c.i_idx = n;
  c.h_items = h_sb[n + 1];
  return c;
}

constexpr uint32_t kFullWarp = 0xFFFFFFFFu;

// A grammar that is known to have no counted repetition: the same tables seen through a type for which the decoding
// of state words below compiles away.  The step kernels exist in both forms and the host picks per batch (C3: the
// decode costs 1.2 us of a 38 us step, although it never finds a count there).
struct PlainGrammarDev : GrammarDev {};
template <typename G> struct HasCounts { static constexpr bool value = true; };
template <> struct HasCounts<PlainGrammarDev> { static constexpr bool value = false; };
template <bool kCounts> struct GrammarAs { typedef GrammarDev type; };
template <> struct GrammarAs<false> { typedef PlainGrammarDev type; };
template <bool kCounts>
__device__ __forceinline__ const typename GrammarAs<kCounts>::type& grammar_as(const GrammarDev& g) { return static_cast<const typename GrammarAs<kCounts>::type&>(g); }

// Counted repetitions (Section 3.6).  rec_of: the record (index into state[], state_first[], entries[]) of an item's
// state word; ordinary states are their own record.
// (`rep_first`: g.rep_first, read once by the caller -- the walks are chains of dependent loads, and the test that almost
// always ends here must not wait for a load of its own)
template <typename G>
__device__ __forceinline__ uint32_t rec_of(const G& g, uint32_t w, uint32_t rep_first) {
  if (!HasCounts<G>::value) return w;
  if (w < rep_first) return w;
  const uint32_t q = w & ((1u << g.rep_shift) - 1u);
  const int done = (int)(w >> g.rep_shift) + 1;
  if (!XG_BOUND((int)q - g.rep_first, g.n_words_states - g.rep_first, kBoundState)) return 0;
  const int4 rs = g.rep_state[q - (uint32_t)g.rep_first];
  const int dl = min(max(rs.y - done, 0), g.rep_depth), dr = max(min(rs.z - done, g.rep_depth), 0);
  return (uint32_t)(rs.x + dl * (g.rep_depth + 1) + dr);
}
template <typename G>
__device__ __forceinline__ uint32_t rec_of(const G& g, uint32_t w) { return rec_of(g, w, (uint32_t)g.rep_first); }
// a state word that belongs to record `rec` (the record itself for ordinary states)
__device__ __forceinline__ uint32_t word_of_record(const GrammarDev& g, int rec) { return g.rec_word ? g.rec_word[rec] : (uint32_t)rec; }
// the state word an edge leads to from the item whose state word is `from`: the packed target, with the count of
// `from` when the edge stays inside a counted rule (kRel), one more when it starts the next iteration (kIter)
template <typename G>
__device__ __forceinline__ uint32_t next_word(const G& g, uint32_t from, uint32_t packed) {
  if (!HasCounts<G>::value) return packed & ~kSelf;
  uint32_t w = packed & kTarget;
  if (packed & kRel) w += (from >> g.rep_shift << g.rep_shift) + ((packed & kIter) ? (1u << g.rep_shift) : 0u);
  return w;
}

// lane -> the index of the first lane whose inclusive prefix exceeds p (the owner of flattened pair p); `n` lanes hold items
__device__ __forceinline__ int owner_of_pair(int incl, int p, int n) {
  int own = 0;
  for (int l = 0; l < n; ++l) own += p >= __shfl_sync(kFullWarp, incl, l) ? 1 : 0;
  return own;
}

__device__ __forceinline__ int warp_inclusive_scan(int x, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(kFullWarp, x, o); if (lane >= o) x += y; }
  return x;
}

// append (ns, no) to the set [start, cnt) unless present; false on overflow
__device__ __forceinline__ bool add_item(uint32_t* st, int32_t* org, int start, int& cnt, int cap, uint32_t ns, int32_t no) {
  for (int q = start; q < cnt; ++q) if (st[q] == ns && org[q] == no) return true;
  if (cnt >= cap) return false;
  st[cnt] = ns; org[cnt] = no; ++cnt;
  return true;
}

// advance every item of chart set `o` that waits for `rule` into the set [start, cnt)
template <typename LsbT, typename G>
__device__ __forceinline__ bool advance_waiters(const G& g, const Chart& c, uint32_t rule, int32_t o, uint32_t* st, int32_t* org,
                                                const LsbT* lsb, int start, int& cnt, int cap) {
  const uint32_t* src_st;
  const int32_t* src_org;
  int b, e;
  if (o < c.i_idx) {
    if (!XG_BOUND(o, c.n + 1, kBoundChartSet)) return true;
    src_st = c.h_st; src_org = c.h_org; b = c.h_sb[o]; e = c.h_sb[o + 1];
    if (!XG_BOUND(e, c.h_items + 1, kBoundChartItem) || !XG_BOUND(b, e + 1, kBoundChartItem)) return true;
  }
  else if (o == c.i_idx) { src_st = c.i_st; src_org = c.i_org; b = 0; e = c.i_cnt; }
  else {
    src_st = st; src_org = org; b = lsb[o - c.i_idx]; e = lsb[o - c.i_idx + 1];
    if (!XG_BOUND(e, cnt + 1, kBoundWalkItem) || !XG_BOUND(b, e + 1, kBoundWalkItem)) return true;
  }
  const uint32_t rep_first = (uint32_t)g.rep_first;
  for (int i = b; i < e; ++i) {
    const uint32_t s2 = src_st[i];
    const int32_t o2 = src_org[i];
    const uint32_t r2 = rec_of(g, s2, rep_first);
    if (!XG_BOUND(r2, g.n_states, kBoundState)) continue;
    const uint4 rec = *reinterpret_cast<const uint4*>(&g.state[r2]);
    const int wait_end = (int)rec.z + (int)(rec.w & 0xFFFFu);
    if (!XG_BOUND(wait_end, g.n_wait_edges + 1, kBoundWaitEdge)) continue;
    // four edges at a time: their loads are issued together, then compared (one at a time, each load would be
    // waited for before the next is even issued)
    for (int w = (int)rec.z; w < wait_end; w += 4) {
      uint2 we[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) we[u] = w + u < wait_end ? g.wait_edge[w + u] : make_uint2(0xFFFFFFFFu, 0u);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (we[u].x != rule) continue;
        if (!add_item(st, org, start, cnt, cap, next_word(g, s2, we[u].y), (we[u].y & kSelf) ? o : o2)) return false;
      }
    }
  }
  return true;
}

// class_bits may point to a shared-memory copy of g.class_bits
template <typename LsbT, typename G>
__device__ __forceinline__ int token_walk(const G& g, const uint32_t* class_bits, const Chart& c, const uint8_t* __restrict__ bytes, int len,
                                          bool own_edges_first, uint32_t* st, int32_t* org, int cap, LsbT* lsb, int* flags, uint32_t* exit_mask) {
  int cnt = 0;
  const uint32_t rep_first = (uint32_t)g.rep_first;
  const uint32_t* cur_st = c.i_st;
  const int32_t* cur_org = c.i_org;
  int cur_b = 0, cur_e = c.i_cnt;
  lsb[0] = 0;
  lsb[1] = 0;
  for (int k = 0; k < len; ++k) {
    const uint32_t byte = bytes[k];
    const uint32_t word = byte >> 5, bit = 1u << (byte & 31);
    const int start = cnt;
    const int self_idx = c.i_idx + k;
    // scan
    for (int i = cur_b; i < cur_e; ++i) {
      const uint32_t s = cur_st[i];
      const int32_t o = cur_org[i];
      const uint32_t sr = rec_of(g, s, rep_first);
      if (!XG_BOUND(sr, g.n_states, kBoundState)) continue;
      const uint4 ra = *reinterpret_cast<const uint4*>(&g.state[sr]);
      const int n_edges = (k == 0 && own_edges_first) ? (int)(ra.y & 0xFFFFu) : (int)(ra.y >> 16);
      if (n_edges == 0) continue;
      if (!XG_BOUND((int)ra.x + n_edges, g.n_scan_edges + 1, kBoundScanEdge)) continue;
      const uint4 rb = *(reinterpret_cast<const uint4*>(&g.state[sr]) + 1);
      // the first edge is inline in the record; the others are fetched four at a time (loads issued together, then tested)
      for (int e = 0; e < n_edges; e += 4) {
        uint2 se[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          se[u] = (e + u == 0) ? make_uint2(rb.z, rb.w) : (e + u < n_edges ? g.scan_edge[(int)ra.x + e + u] : make_uint2(kLiteral | 0x100u, 0u));
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (e + u >= n_edges) break;
          if (!(se[u].x & kLiteral) && !XG_BOUND(se[u].x, g.n_classes, kBoundClass)) continue;
          const bool hit = (se[u].x & kLiteral) ? ((se[u].x & 0x1FFu) == byte) : ((class_bits[se[u].x * 8 + word] & bit) != 0);
          if (hit && !add_item(st, org, start, cnt, cap, next_word(g, s, se[u].y), (se[u].y & kSelf) ? self_idx : o)) { *flags |= kWalkOverflow; return k; }
        }
      }
    }
    if (cnt == start) return k;
    // complete (cascades through the growing set)
    for (int q = start; q < cnt; ++q) {
      const uint32_t qr = rec_of(g, st[q], rep_first);
      if (!XG_BOUND(qr, g.n_states, kBoundState)) continue;
      const uint32_t info = g.state[qr].info;
      if (!(info >> 31)) continue;
      const int32_t o = org[q];
      if (o < 0) {
        if (k + 1 < len) { *flags |= kWalkUncertain; if (exit_mask && k + 1 < 32) *exit_mask |= 1u << (k + 1); }
        continue;
      }
      if (!advance_waiters(g, c, info & 0x7FFFFFFFu, o, st, org, lsb, start, cnt, cap)) { *flags |= kWalkOverflow; return k; }
    }
    cur_st = st; cur_org = org; cur_b = start; cur_e = cnt;
    lsb[k + 2] = (LsbT)cnt;
  }
  return len;
}

// byte-class bitsets staged in shared memory when they fit (the hottest table of a walk)
constexpr int kSharedClasses = 128;     // (the grammars of all workloads here have at most 124 classes)
__device__ __forceinline__ const uint32_t* stage_class_bits(const GrammarDev& g, uint32_t* sh) {
  if (g.n_classes > kSharedClasses) return g.class_bits;
  for (int i = threadIdx.x; i < g.n_classes * 8; i += blockDim.x) sh[i] = g.class_bits[i];
  return sh;
}

// ------------------------------------------------------------------------------------------
// Cache build (Section 3.4; appendix on the adaptive token mask cache): classify every
// (scannable state, token) pair.  grid.y = position, grid.x * block = token rank (trie order).
// Accepted and uncertain bits are scattered into id-ordered rows; the uncertain bits are also
// ballot-packed in rank order (the order later walks use).
// ------------------------------------------------------------------------------------------
// A block classifies one chunk of kClassifyChunk tokens of one position.  Only tokens whose first byte the position's
// own edges can take are ever looked at: in trie order the tokens that start with byte b are the ranks
// [first_rank[b], first_rank[b + 1]), so the position's viable tokens are a union of at most 256 rank ranges, and the
// host lists, per position, as many chunks as those ranges hold tokens (work[i] = (position, chunk)).  Everything
// else is rejected without being touched: the rows are zeroed beforehand.
constexpr int kClassifyChunk = 2048;

// kCount: also add up the bytes the walks consume (viable trie nodes visited, without any sharing between tokens)
// into *visits -- the work the classification actually does, as opposed to the (position, token) pairs it decides.
// kCounts: the grammar has counted repetitions (otherwise the decoding of state words compiles away)
template <bool kCount, bool kCounts>
__global__ void __launch_bounds__(256)
classify_kernel(GrammarDev g_, VocabDev v, const int32_t* __restrict__ positions, const int2* __restrict__ work,
                uint32_t* __restrict__ acc_id, uint32_t* __restrict__ unc_id, uint32_t* __restrict__ unc_rank,
                int2* __restrict__ overflow, int* __restrict__ overflow_count, int overflow_cap, unsigned long long* __restrict__ visits) {
  __shared__ uint32_t sh_st[1];
  __shared__ int32_t sh_org[1];
  __shared__ uint32_t sh_class[kSharedClasses * 8];
  __shared__ uint32_t sh_first[8];          // bytes the position's own edges can take
  __shared__ int sh_cum[257];               // sh_cum[b]: viable tokens whose first byte is below b
  const typename GrammarAs<kCounts>::type& g = grammar_as<kCounts>(g_);
  const int pos = work[blockIdx.x].x, chunk = work[blockIdx.x].y;
  const int state = positions[pos];
  if (threadIdx.x < 8) {
    const StateRec rec = g.state[state];
    uint32_t w = 0;
    for (int e = 0; e < (int)(rec.n_own_n_scan & 0xFFFFu); ++e) {
      const uint32_t code = e == 0 ? rec.edge0_class : g.scan_edge[rec.scan_begin + e].x;
      if (code & kLiteral) w |= ((code & 0xFFu) >> 5) == threadIdx.x ? 1u << (code & 31u) : 0u;
      else w |= g.class_bits[code * 8 + threadIdx.x];
    }
    sh_first[threadIdx.x] = w;
  }
  if (threadIdx.x == 0) { sh_st[0] = word_of_record(g, state); sh_org[0] = -1; }
  const uint32_t* class_bits = stage_class_bits(g, sh_class);
  __syncthreads();
  {   // inclusive scan of the 256 range lengths (thread b holds byte b), shifted into sh_cum[b + 1]
    const int b = (int)threadIdx.x;
    int x = ((sh_first[b >> 5] >> (b & 31)) & 1u) ? (int)(v.first_rank[b + 1] - v.first_rank[b]) : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xFFFFFFFFu, x, o); if ((b & 31) >= o) x += y; }
    __shared__ int warp_sum[8];
    if ((b & 31) == 31) warp_sum[b >> 5] = x;
    __syncthreads();
    int base = 0;
    for (int w = 0; w < (b >> 5); ++w) base += warp_sum[w];
    sh_cum[b + 1] = base + x;
    if (b == 0) sh_cum[0] = 0;
  }
  __syncthreads();
  const int total = sh_cum[256];
  for (int i = 0; i < kClassifyChunk / 256; ++i) {
    const int idx = chunk * kClassifyChunk + i * 256 + (int)threadIdx.x;        // the idx-th viable token of this position
    int cls = 0, walked = 0, rank = -1;
    if (idx < total) {
      int lo = 0, hi = 256;                   // the first byte whose range holds idx: sh_cum[lo] <= idx < sh_cum[lo + 1]
      while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (sh_cum[mid] <= idx) lo = mid; else hi = mid; }
      rank = (int)v.first_rank[lo] + (idx - sh_cum[lo]);
    }
    if (rank >= 0 && XG_BOUND(rank, v.vocab_size, kBoundTokenRank) && !v.never[rank]) {
      const uint32_t off = v.offset[rank];
      const int len = (int)(v.offset[rank + 1] - off);
      int flags = 0;
      int consumed = 0;
      if (len > kFastMaxBytes) flags = kWalkOverflow;
      else {
        uint32_t st[kFastCap];
        int32_t org[kFastCap];
        int16_t lsb[kFastMaxBytes + 2];
        Chart c;
        c.h_st = nullptr; c.h_org = nullptr; c.h_sb = nullptr; c.n = -1; c.h_items = 0;
        c.i_st = sh_st; c.i_org = sh_org; c.i_cnt = 1; c.i_idx = 0;
        consumed = token_walk<int16_t>(g, class_bits, c, v.bytes + off, len, true, st, org, kFastCap, lsb, &flags, nullptr);
        walked = consumed;
      }
      if (flags & kWalkOverflow) {
        int slot = atomicAdd(overflow_count, 1);
        if (slot < overflow_cap) overflow[slot] = make_int2(pos, rank);
      } else if (consumed == len) cls = 1;
      else if (flags & kWalkUncertain) cls = 2;
      if (cls) {
        const int id = v.rank_to_id[rank];
        uint32_t* row = (cls == 1 ? acc_id : unc_id) + (size_t)pos * v.n_words;
        atomicOr(&row[id >> 5], 1u << (id & 31));
        if (cls == 2) atomicOr(&unc_rank[(size_t)pos * v.n_words + (rank >> 5)], 1u << (rank & 31));
      }
    }
    if (kCount) {
      const int sum = __reduce_add_sync(0xFFFFFFFFu, walked);
      if ((threadIdx.x & 31) == 0 && sum) atomicAdd(visits, (unsigned long long)sum);
    }
  }
}

// exact fallback for the pairs whose walk did not fit the fast path's fixed arrays
__global__ void classify_slow_kernel(GrammarDev g, VocabDev v, const int32_t* __restrict__ positions,
                                     const int2* __restrict__ pairs, int n_pairs, uint32_t* scratch_st, int32_t* scratch_org,
                                     int32_t* scratch_lsb, uint32_t* acc_id, uint32_t* unc_id, uint32_t* unc_rank,
                                     int* __restrict__ failed) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_pairs) return;
  const int pos = pairs[i].x, rank = pairs[i].y;
  uint32_t h_st = word_of_record(g, positions[pos]);
  int32_t h_org = -1;
  Chart c;
  c.h_st = nullptr; c.h_org = nullptr; c.h_sb = nullptr; c.n = -1; c.h_items = 0;
  c.i_st = &h_st; c.i_org = &h_org; c.i_cnt = 1; c.i_idx = 0;
  const uint32_t off = v.offset[rank];
  const int len = (int)(v.offset[rank + 1] - off);
  if (len > kSlowMaxBytes) { atomicExch(failed, 1); return; }
  int flags = 0;
  int consumed = token_walk<int32_t>(g, g.class_bits, c, v.bytes + off, len, true, scratch_st + (size_t)i * kSlowCap,
                                     scratch_org + (size_t)i * kSlowCap, kSlowCap, scratch_lsb + (size_t)i * (kSlowMaxBytes + 2), &flags, nullptr);
  if (flags & kWalkOverflow) { atomicExch(failed, 1); return; }
  int cls = consumed == len ? 1 : ((flags & kWalkUncertain) ? 2 : 0);
  if (!cls) return;
  const int id = v.rank_to_id[rank];
  uint32_t* row = (cls == 1 ? acc_id : unc_id) + (size_t)pos * v.n_words;
  atomicOr(&row[id >> 5], 1u << (id & 31));
  if (cls == 2) atomicOr(&unc_rank[(size_t)pos * v.n_words + (rank >> 5)], 1u << (rank & 31));
}

// ------------------------------------------------------------------------------------------
// Adaptive pack (Section 3.3 "adaptive storage"): per position count, choose the smallest of
// accepted list / rejected list / bitset, exclusive-scan the sizes, compact.
// ------------------------------------------------------------------------------------------
struct PackPlan {
  long long offset_words;   // into the arena
  int32_t kind, n_list, n_acc, n_unc;
};

__device__ __forceinline__ int block_reduce_sum(int x, int* sh) {
  for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xFFFFFFFFu, x, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = x;
  __syncthreads();
  int total = 0;
  const int nw = (blockDim.x + 31) >> 5;
  for (int i = 0; i < nw; ++i) total += sh[i];
  __syncthreads();
  return total;
}

__global__ void __launch_bounds__(256)
count_kernel(const uint32_t* __restrict__ acc_id, const uint32_t* __restrict__ unc_id, int n_words, int2* __restrict__ counts) {
  __shared__ int sh[8];
  const size_t base = (size_t)blockIdx.x * n_words;
  int a = 0, u = 0;
  for (int w = threadIdx.x; w < n_words; w += blockDim.x) { a += __popc(acc_id[base + w]); u += __popc(unc_id[base + w]); }
  a = block_reduce_sum(a, sh);
  u = block_reduce_sum(u, sh);
  if (threadIdx.x == 0) counts[blockIdx.x] = make_int2(a, u);
}

// one block: kinds, sizes and arena offsets for all positions of the batch
__global__ void __launch_bounds__(1024)
plan_kernel(const int2* __restrict__ counts, int n_pos, int vocab_size, int n_words, PackPlan* __restrict__ plan, long long* __restrict__ total_words) {
  __shared__ long long sums[1024];
  const int per = (n_pos + blockDim.x - 1) / blockDim.x;
  const int lo = min(n_pos, (int)threadIdx.x * per), hi = min(n_pos, lo + per);
  long long local = 0;
  for (int p = lo; p < hi; ++p) {
    const int na = counts[p].x, nu = counts[p].y, nr = vocab_size - na - nu;
    int kind = 0, n_list = na;                       // ties: accepted list < rejected list < bitset
    if (nr < n_list) { kind = 1; n_list = nr; }
    if (n_words < n_list) { kind = 2; n_list = 0; }
    plan[p].kind = kind; plan[p].n_list = n_list; plan[p].n_acc = na; plan[p].n_unc = nu;
    local += (kind == 2 ? n_words : n_list) + 4LL * nu;
  }
  sums[threadIdx.x] = local;
  __syncthreads();
  for (int off = 1; off < (int)blockDim.x; off <<= 1) {
    long long add = (int)threadIdx.x >= off ? sums[threadIdx.x - off] : 0;
    __syncthreads();
    sums[threadIdx.x] += add;
    __syncthreads();
  }
  long long run = sums[threadIdx.x] - local;
  for (int p = lo; p < hi; ++p) {
    plan[p].offset_words = run;
    run += (plan[p].kind == 2 ? n_words : plan[p].n_list) + 4LL * plan[p].n_unc;
  }
  if (threadIdx.x == blockDim.x - 1) *total_words = sums[threadIdx.x];
}

// ascending positions of the set bits of word_fn(w), w in [0, n_words), written to out
template <typename F>
__device__ __forceinline__ void compact_bits(F word_fn, int n_words, uint32_t* __restrict__ out, int* sh_scan) {
  const int per = (n_words + blockDim.x - 1) / blockDim.x;
  const int lo = min(n_words, (int)threadIdx.x * per), hi = min(n_words, lo + per);
  int mine = 0;
  for (int w = lo; w < hi; ++w) mine += __popc(word_fn(w));
  sh_scan[threadIdx.x] = mine;
  __syncthreads();
  for (int off = 1; off < (int)blockDim.x; off <<= 1) {
    int add = (int)threadIdx.x >= off ? sh_scan[threadIdx.x - off] : 0;
    __syncthreads();
    sh_scan[threadIdx.x] += add;
    __syncthreads();
  }
  int at = sh_scan[threadIdx.x] - mine;
  for (int w = lo; w < hi; ++w) {
    uint32_t bits = word_fn(w);
    while (bits) { int j = __ffs(bits) - 1; bits &= bits - 1; out[at++] = (uint32_t)(w * 32 + j); }
  }
  __syncthreads();
}

__global__ void __launch_bounds__(256)
pack_kernel(const uint32_t* __restrict__ acc_id, const uint32_t* __restrict__ unc_id, const uint32_t* __restrict__ unc_rank,
            const PackPlan* __restrict__ plan, int vocab_size, int n_words, uint32_t* __restrict__ arena, EntryDev* __restrict__ entries,
            const int* __restrict__ go) {
  __shared__ int sh_scan[256];
  if (go && !*go) return;                 // a just-in-time build that found no room (see jit_reserve_kernel)
  const int p = blockIdx.x;
  const PackPlan pl = plan[p];
  const uint32_t* a = acc_id + (size_t)p * n_words;
  const uint32_t* u = unc_id + (size_t)p * n_words;
  const uint32_t* ur = unc_rank + (size_t)p * n_words;
  uint32_t* data = arena + pl.offset_words;
  const int n_data = pl.kind == 2 ? n_words : pl.n_list;
  uint32_t* out_uid = data + n_data;
  uint32_t* out_urank = out_uid + pl.n_unc;
  if (pl.kind == 2) {
    for (int w = threadIdx.x; w < n_words; w += blockDim.x) data[w] = a[w];
  } else if (pl.kind == 0) {
    compact_bits([&](int w) { return a[w]; }, n_words, data, sh_scan);
  } else {
    const uint32_t tail = (vocab_size & 31) ? ((1u << (vocab_size & 31)) - 1) : 0xFFFFFFFFu;
    compact_bits([&](int w) { uint32_t x = ~(a[w] | u[w]); return w == n_words - 1 ? (x & tail) : x; }, n_words, data, sh_scan);
  }
  compact_bits([&](int w) { return u[w]; }, n_words, out_uid, sh_scan);
  compact_bits([&](int w) { return ur[w]; }, n_words, out_urank, sh_scan);
  if (threadIdx.x == 0) {
    EntryDev e;
    e.data = data; e.unc_id = out_uid; e.unc_rank = out_urank; e.unc_exit = out_urank + pl.n_unc;
    e.unc_info = out_urank + 2 * (size_t)pl.n_unc;
    e.kind = pl.kind; e.n_list = pl.n_list; e.n_unc = pl.n_unc; e.n_acc = pl.n_acc;
    e.chk_rank = e.unc_rank; e.chk_exit = e.unc_exit; e.chk_info = e.unc_info; e.n_chk = pl.n_unc; e.pad2 = 0;
    entries[p] = e;
  }
}

// what a token (bytes at `off`, `len` of them) has left at the first exit of `exits`: see EntryDev::unc_info
__device__ __forceinline__ uint32_t first_exit_info(const VocabDev& v, uint32_t off, int len, uint32_t exits) {
  if (!exits) return 0;
  const int at = __ffs(exits) - 1;
  const uint32_t b1 = v.bytes[off + at], b2 = at + 1 < len ? v.bytes[off + at + 1] : 0u;
  return b1 | (b2 << 8) | ((uint32_t)min(len - at, 255) << 16);
}

// For every uncertain token of every packed entry: the byte offsets at which the token leaves
// the entry's rule (bit j = after j bytes).  The run-time check restarts there instead of
// re-walking the part of the token that the cache already decided.  0 = unknown (walk in full).
template <bool kCounts>
__global__ void __launch_bounds__(256)
exit_kernel(GrammarDev g_, VocabDev v, const int32_t* __restrict__ positions, const EntryDev* __restrict__ entries, const int* __restrict__ go) {
  if (go && !*go) return;
  const typename GrammarAs<kCounts>::type& g = grammar_as<kCounts>(g_);
  __shared__ uint32_t sh_st[1];
  __shared__ int32_t sh_org[1];
  __shared__ uint32_t sh_class[kSharedClasses * 8];
  const int p = blockIdx.x;
  const EntryDev e = entries[p];
  if (threadIdx.x == 0) { sh_st[0] = word_of_record(g, positions[p]); sh_org[0] = -1; }
  const uint32_t* class_bits = stage_class_bits(g, sh_class);
  __syncthreads();
  uint32_t* out = const_cast<uint32_t*>(e.unc_exit);
  uint32_t* out_info = const_cast<uint32_t*>(e.unc_info);
  for (int k = threadIdx.x; k < e.n_unc; k += blockDim.x) {
    const int rank = (int)e.unc_rank[k];
    const uint32_t off = v.offset[rank];
    const int len = (int)(v.offset[rank + 1] - off);
    uint32_t mask = 0;
    if (len <= kFastMaxBytes) {
      uint32_t st[kFastCap];
      int32_t org[kFastCap];
      int16_t lsb[kFastMaxBytes + 2];
      int flags = 0;
      Chart c;
      c.h_st = nullptr; c.h_org = nullptr; c.h_sb = nullptr; c.n = -1; c.h_items = 0;
      c.i_st = sh_st; c.i_org = sh_org; c.i_cnt = 1; c.i_idx = 0;
      token_walk<int16_t>(g, class_bits, c, v.bytes + off, len, true, st, org, kFastCap, lsb, &flags, &mask);
      if (flags & kWalkOverflow) mask = 0;
    }
    out[k] = mask;
    out_info[k] = first_exit_info(v, off, len, mask);
  }
}

// Lookahead (Section 3.3): narrow each entry's uncertain list with the grammar's follow set of
// the entry's rule.  An exit survives iff the byte after it can follow the rule somewhere in this
// grammar; a token survives iff it keeps an exit (tokens without an exit record are kept).
// First pass counts, second pass compacts in list order.
__device__ __forceinline__ uint32_t narrow_exits(const VocabDev& v, const uint32_t* __restrict__ follow, int rank, uint32_t exits) {
  if (exits == 0) return 0;
  const uint32_t off = v.offset[rank];
  uint32_t keep = 0;
  for (uint32_t left = exits; left; left &= left - 1) {
    const int at = __ffs(left) - 1;
    const uint32_t byte = v.bytes[off + at];
    if ((follow[byte >> 5] >> (byte & 31)) & 1u) keep |= 1u << at;
  }
  return keep;
}

__global__ void __launch_bounds__(256)
lookahead_count_kernel(GrammarDev g, VocabDev v, const int32_t* __restrict__ states, int32_t* __restrict__ counts, const int* __restrict__ go) {
  __shared__ int sh[8];
  if (go && !*go) return;
  const int q = states[blockIdx.x];
  const EntryDev e = g.entries[q];
  const uint32_t* follow = g.rule_follow + (size_t)(g.state[q].info & 0x7FFFFFFFu) * 8;
  int mine = 0;
  for (int k = threadIdx.x; k < e.n_unc; k += blockDim.x) {
    const uint32_t exits = e.unc_exit[k];
    mine += (exits == 0 || narrow_exits(v, follow, (int)e.unc_rank[k], exits) != 0) ? 1 : 0;
  }
  mine = block_reduce_sum(mine, sh);
  if (threadIdx.x == 0) counts[blockIdx.x] = mine;
}

__global__ void __launch_bounds__(256)
lookahead_compact_kernel(GrammarDev g, VocabDev v, const int32_t* __restrict__ states, const long long* __restrict__ offsets,
                         const int32_t* __restrict__ counts, uint32_t* __restrict__ arena, const int* __restrict__ go) {
  __shared__ int sh_scan[256];
  if (go && !*go) return;
  const int q = states[blockIdx.x];
  const EntryDev e = g.entries[q];
  const uint32_t* follow = g.rule_follow + (size_t)(g.state[q].info & 0x7FFFFFFFu) * 8;
  const int n_out = counts[blockIdx.x];
  uint32_t* out_rank = arena + offsets[blockIdx.x];
  uint32_t* out_exit = out_rank + n_out;
  uint32_t* out_info = out_exit + n_out;
  const int per = (e.n_unc + blockDim.x - 1) / blockDim.x;
  const int lo = min(e.n_unc, (int)threadIdx.x * per), hi = min(e.n_unc, lo + per);
  int mine = 0;
  for (int k = lo; k < hi; ++k) {
    const uint32_t exits = e.unc_exit[k];
    mine += (exits == 0 || narrow_exits(v, follow, (int)e.unc_rank[k], exits) != 0) ? 1 : 0;
  }
  sh_scan[threadIdx.x] = mine;
  __syncthreads();
  for (int off = 1; off < (int)blockDim.x; off <<= 1) {
    int add = (int)threadIdx.x >= off ? sh_scan[threadIdx.x - off] : 0;
    __syncthreads();
    sh_scan[threadIdx.x] += add;
    __syncthreads();
  }
  int at = sh_scan[threadIdx.x] - mine;
  for (int k = lo; k < hi; ++k) {
    const uint32_t exits = e.unc_exit[k];
    const int rank = (int)e.unc_rank[k];
    const uint32_t keep = narrow_exits(v, follow, rank, exits);
    if (exits != 0 && keep == 0) continue;
    out_rank[at] = (uint32_t)rank;
    out_exit[at] = keep;
    out_info[at] = first_exit_info(v, v.offset[rank], (int)(v.offset[rank + 1] - v.offset[rank]), keep);
    ++at;
  }
}

// ------------------------------------------------------------------------------------------
// Just-in-time cache build (Section 3.5): the same classify / count / plan / pack / exit kernels,
// enqueued between decode steps without a host round trip.  The two things the host does in the
// compile-time build -- sizing the arena from the plan's total and checking for walks that left
// the fast path -- happen here on the device.
// ------------------------------------------------------------------------------------------
// result[0]: 1 = go on, 0 = stop (result[1] says why: 1 = no room in the arena, 2 = a token walk
// needs the exact slow path, which only the host can set up)
__global__ void jit_reserve_kernel(PackPlan* __restrict__ plan, int n_pos, const long long* __restrict__ total_words,
                                   unsigned long long* __restrict__ arena_used, long long arena_cap,
                                   const int* __restrict__ overflow_count, int* __restrict__ result) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  result[0] = 0; result[1] = 0;
  if (*overflow_count > 0) { result[1] = 2; return; }
  const unsigned long long need = (unsigned long long)max(*total_words, 1LL);
  const unsigned long long base = atomicAdd(arena_used, need);
  if (base + need > (unsigned long long)arena_cap) { result[1] = 1; return; }
  for (int p = 0; p < n_pos; ++p) plan[p].offset_words += (long long)base;
  result[0] = 1;
}

// Make freshly built entries visible to the fill kernels: every state whose class representative
// was built takes the representative's entry.  `built_state` / `built_entry`: the n entries.
__global__ void __launch_bounds__(256)
jit_publish_kernel(EntryDev* __restrict__ entries, const int32_t* __restrict__ rep, int n_states,
                   const int32_t* __restrict__ built_state, const EntryDev* __restrict__ built_entry, int n, const int* __restrict__ go) {
  if (go && !*go) return;
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= n_states) return;
  const int r = rep[s];
  for (int k = 0; k < n; ++k)
    if (built_state[k] == r) { entries[s] = built_entry[k]; return; }
}

// Lookahead narrowing of just-built entries (Section 3.3), again without the host: room for the
// narrowed check lists comes from the same arena.  If there is none the entries simply keep their
// whole uncertain lists as check lists.
__global__ void jit_reserve_lists_kernel(const int32_t* __restrict__ counts, int n, long long* __restrict__ offsets,
                                         unsigned long long* __restrict__ arena_used, long long arena_cap,
                                         const int* __restrict__ go, int* __restrict__ go_lists) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  *go_lists = 0;
  if (!*go) return;
  unsigned long long need = 1;
  for (int k = 0; k < n; ++k) need += 3ull * counts[k];
  const unsigned long long base = atomicAdd(arena_used, need);
  if (base + need > (unsigned long long)arena_cap) return;
  long long run = (long long)base;
  for (int k = 0; k < n; ++k) { offsets[k] = run; run += 3LL * counts[k]; }
  *go_lists = 1;
}

__global__ void __launch_bounds__(256)
jit_patch_lists_kernel(EntryDev* __restrict__ entries, const int32_t* __restrict__ rep, int n_states, const int32_t* __restrict__ built_state,
                       const int32_t* __restrict__ counts, const long long* __restrict__ offsets, const uint32_t* __restrict__ arena, int n,
                       const int* __restrict__ go_lists) {
  if (!*go_lists) return;
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= n_states) return;
  const int r = rep[s];
  for (int k = 0; k < n; ++k)
    if (built_state[k] == r) {
      EntryDev& e = entries[s];
      e.chk_rank = arena + offsets[k];
      e.chk_exit = e.chk_rank + counts[k];
      e.chk_info = e.chk_exit + counts[k];
      e.n_chk = counts[k];
      return;
    }
}

// ------------------------------------------------------------------------------------------
// matcher state
// ------------------------------------------------------------------------------------------
// is the root rule complete in the current set (EOS allowed)?
template <typename G>
__device__ __forceinline__ bool root_complete(const MatcherDev& m, const G& g) {
  if (m.n_sets == 1 && g.root_nullable) return true;
  const int n = m.n_sets - 1;
  for (int i = m.set_begin[n]; i < m.set_begin[n + 1]; ++i) {
    if (m.item_origin[i] != 0) continue;
    const uint32_t info = g.state[rec_of(g, m.item_state[i])].info;
    if ((info >> 31) && (info & 0x7FFFFFFFu) == (uint32_t)g.root_rule) return true;
  }
  return false;
}

// Build the step plan of the request's current set, by one warp.  The entries are listed with one lane per (item of
// the set, entry of its gather list) pair, so that the table lookups behind every pair -- the item's record, the gather
// entry, the cache entry's header -- are three rounds of loads for the whole set; the lists themselves are kept in
// registers, one slot per lane, and a pair is added to them by a compare in every lane and a vote.  Then one lane per
// entry completes that entry's rule into its continuation set.
template <typename G>
__device__ __forceinline__ void prepare_plan(MatcherDev& m, const G& g, int lane) {
  StepPlan& p = *m.plan;
  const int n = m.n_sets - 1;
  const uint32_t rep_first = (uint32_t)g.rep_first;
  const Chart hist = chart_of_history(m.item_state, m.item_origin, m.set_begin, n);
  int n_merge = 0, n_check = 0, n_missing = 0, overflow = 0;       // (the same in every lane)
  int merge_lo = -1, merge_hi = -1;           // slots lane and lane + 32 of the merge list
  int check_q = -1, check_o = 0, check_n = 0; // slot lane of the check list: state, origin, candidates
  int missing_q = -1;                         // slot lane of the missing list (lanes below kPlanMissingMax)
  bool root_done = m.n_sets == 1 && g.root_nullable;
  static_assert(kPlanMergeMax == 64 && kPlanCheckMax == 32 && kPlanMissingMax <= 32, "one or two list slots per lane");
  for (int base = 0; base < hist.i_cnt && !overflow; base += 32) {
    const int n_here = min(32, hist.i_cnt - base);
    const bool have = lane < n_here;
    const uint32_t s = have ? rec_of(g, hist.i_st[base + lane], rep_first) : 0u;
    const int32_t o = have ? hist.i_org[base + lane] : 0;
    int gather_begin = 0, n_gather = 0;
    if (have && XG_BOUND(s, g.n_states, kBoundState)) {
      const uint4 ra = *reinterpret_cast<const uint4*>(&g.state[s]), rb = *(reinterpret_cast<const uint4*>(&g.state[s]) + 1);
      gather_begin = (int)rb.x; n_gather = (int)(ra.w >> 16);
      if (!XG_BOUND(gather_begin + n_gather, g.n_gather + 1, kBoundGather)) n_gather = 0;
      // EOS is allowed iff the root rule is complete with origin 0
      root_done = root_done || (o == 0 && (rb.y >> 31) && (rb.y & 0x7FFFFFFFu) == (uint32_t)g.root_rule);
    }
    const int incl = warp_inclusive_scan(n_gather, lane);
    const int total = __shfl_sync(kFullWarp, incl, 31);
    for (int p0 = 0; p0 < total && !overflow; p0 += 32) {
      const int pi = p0 + lane;
      const int own = min(owner_of_pair(incl, pi, n_here), 31);
      const int first = __shfl_sync(kFullWarp, incl - n_gather, own), gb = __shfl_sync(kFullWarp, gather_begin, own);
      const int32_t o_own = __shfl_sync(kFullWarp, o, own);
      int q = -1, origin = 0, kind = 0, n_chk = 0;
      if (pi < total) {
        const int code = g.gather_state[gb + (pi - first)];
        q = code & 0x7FFFFFFF;
        origin = code < 0 ? n : o_own;                       // predicted start states begin here
        if (XG_BOUND(q, g.n_states, kBoundEntry)) { kind = g.entries[q].kind; n_chk = g.entries[q].n_chk; } else q = -1;
      }
      uint32_t todo = __ballot_sync(kFullWarp, q >= 0);
      while (todo && !overflow) {                            // the pairs in order, each decided by all lanes at once
        const int h = __ffs(todo) - 1;
        todo &= todo - 1;
        const int qh = __shfl_sync(kFullWarp, q, h), oh = __shfl_sync(kFullWarp, origin, h);
        const int kh = __shfl_sync(kFullWarp, kind, h), nh = __shfl_sync(kFullWarp, n_chk, h);
        if (kh == kEntryNotBuilt) {                          // a just-in-time grammar has not built this entry yet
          if (!__any_sync(kFullWarp, lane < min(n_missing, kPlanMissingMax) && missing_q == qh)) {
            if (lane == n_missing) missing_q = qh;           // (beyond kPlanMissingMax only counted)
            ++n_missing;
          }
          continue;
        }
        if (!__any_sync(kFullWarp, (lane < n_merge && merge_lo == qh) || (lane + 32 < n_merge && merge_hi == qh))) {
          if (n_merge == kPlanMergeMax) { overflow = 1; break; }
          if (lane == (n_merge & 31)) { if (n_merge < 32) merge_lo = qh; else merge_hi = qh; }
          ++n_merge;
        }
        if (nh == 0) continue;
        if (__any_sync(kFullWarp, lane < n_check && check_q == qh && check_o == oh)) continue;
        if (n_check == kPlanCheckMax) { overflow = 1; break; }
        if (lane == n_check) { check_q = qh; check_o = oh; check_n = nh; }
        ++n_check;
      }
    }
  }
  if (lane < n_merge) p.merge_state[lane] = merge_lo;
  if (lane + 32 < n_merge) p.merge_state[lane + 32] = merge_hi;
  if (lane < min(n_missing, kPlanMissingMax)) p.missing_state[lane] = missing_q;
  const int cum = warp_inclusive_scan(lane < n_check ? check_n : 0, lane);
  if (lane < n_check) { p.check_state[lane] = check_q; p.check_origin[lane] = check_o; p.check_cum[lane + 1] = cum; }
  root_done = __any_sync(kFullWarp, root_done);
  if (lane == 0) {
    p.check_cum[0] = 0;
    p.n_merge = n_merge; p.n_check = n_check; p.overflow = overflow; p.n_missing = n_missing;
    p.eos_ok = root_done ? 1 : 0;
  }
  __syncwarp();
  // continuation set of every entry: complete rule(q) started at its origin, with cascades
  bool bad = false;
  for (int e = lane; e < n_check; e += 32) {
    uint32_t* st = p.cont_st[e];
    int32_t* org = p.cont_org[e];
    int cnt = 0;
    int16_t no_local[2] = {0, 0};
    bool ok = advance_waiters(g, hist, g.state[p.check_state[e]].info & 0x7FFFFFFFu, p.check_origin[e], st, org, no_local, 0, cnt, kContCap);
    for (int q = 0; ok && q < cnt; ++q) {
      const uint32_t info = g.state[rec_of(g, st[q], rep_first)].info;
      if (info >> 31) ok = advance_waiters(g, hist, info & 0x7FFFFFFFu, org[q], st, org, no_local, 0, cnt, kContCap);
    }
    if (!ok) { bad = true; cnt = 0; }
    p.cont_cnt[e] = cnt;
    uint4 fa = make_uint4(0, 0, 0, 0), fb = make_uint4(0, 0, 0, 0);
    for (int q = 0; q < cnt; ++q) {
      const uint4* sf = reinterpret_cast<const uint4*>(g.state_first + (size_t)rec_of(g, st[q], rep_first) * 8);
      const uint4 a = sf[0], c = sf[1];
      fa.x |= a.x; fa.y |= a.y; fa.z |= a.z; fa.w |= a.w;
      fb.x |= c.x; fb.y |= c.y; fb.z |= c.z; fb.w |= c.w;
    }
    uint4* out = reinterpret_cast<uint4*>(p.cont_first[e]);
    out[0] = fa; out[1] = fb;
  }
  if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) p.overflow = 1;
}

// the matcher's initial state: one item, the root rule's start state at origin 0 (lane 0 writes)
__device__ __forceinline__ void matcher_restart(MatcherDev& m, const GrammarDev& g) {
  m.item_state[0] = (uint32_t)g.root_start;
  m.item_origin[0] = 0;
  m.set_begin[0] = 0;
  m.set_begin[1] = 1;
  m.n_sets = 1;
  m.n_items = 1;
  m.terminated = 0;
}

__global__ void matcher_reset_kernel(MatcherDev* m) {      // one warp
  if (blockIdx.x != 0 || threadIdx.x >= 32) return;
  if (threadIdx.x == 0) matcher_restart(*m, *m->grammar);
  __syncwarp();
  prepare_plan(*m, *m->grammar, threadIdx.x);
}

// ------------------------------------------------------------------------------------------
// The token walk by a whole warp (the sampled token of one request: nothing else to do at that moment, and its
// latency is the step's).  The same scan / complete as token_walk, but the lanes share every round of loads: in the
// scan each lane takes one (item, scan edge) pair of the current set -- the records of all items, then all edges,
// then the class words they need are each one round trip, however many edges a state has (a string-body state has
// about ten) --, a ballot collects the hits, and in a completion each lane takes one (waiting item, wait edge)
// pair of the origin set.  Sets live in the warp's shared-memory scratch (st, org: `cap` items; lsb as in
// token_walk).  All 32 lanes must call; the result is the same in every lane.
// ------------------------------------------------------------------------------------------

// append (ns, no) to the set [start, cnt) unless present (same arguments in every lane); false on overflow
__device__ __forceinline__ bool warp_add_item(uint32_t* st, int32_t* org, int start, int& cnt, int cap, uint32_t ns, int32_t no, int lane) {
  bool dup = false;
  for (int q = start + lane; q < cnt; q += 32) dup = dup || (st[q] == ns && org[q] == no);
  if (__any_sync(kFullWarp, dup)) return true;
  if (cnt >= cap) return false;
  if (lane == 0) { st[cnt] = ns; org[cnt] = no; }
  ++cnt;
  __syncwarp();
  return true;
}

// advance every item of chart set `o` that waits for `rule` into the set [start, cnt)
template <typename LsbT, typename G>
__device__ __forceinline__ bool warp_advance_waiters(const G& g, const Chart& c, uint32_t rule, int32_t o, uint32_t* st, int32_t* org,
                                                     const LsbT* lsb, int start, int& cnt, int cap, int lane) {
  const uint32_t* src_st;
  const int32_t* src_org;
  int b, e;
  if (o < c.i_idx) {
    if (!XG_BOUND(o, c.n + 1, kBoundChartSet)) return true;
    src_st = c.h_st; src_org = c.h_org; b = c.h_sb[o]; e = c.h_sb[o + 1];
    if (!XG_BOUND(e, c.h_items + 1, kBoundChartItem) || !XG_BOUND(b, e + 1, kBoundChartItem)) return true;
  }
  else if (o == c.i_idx) { src_st = c.i_st; src_org = c.i_org; b = 0; e = c.i_cnt; }
  else {
    src_st = st; src_org = org; b = lsb[o - c.i_idx]; e = lsb[o - c.i_idx + 1];
    if (!XG_BOUND(e, cnt + 1, kBoundWalkItem) || !XG_BOUND(b, e + 1, kBoundWalkItem)) return true;
  }
  const uint32_t rep_first = (uint32_t)g.rep_first;
  for (int base = b; base < e; base += 32) {
    const int n_here = min(32, e - base);
    const bool have = lane < n_here;
    const uint32_t s2 = have ? src_st[base + lane] : 0u;
    const int32_t o2 = have ? src_org[base + lane] : 0;
    uint4 rec = make_uint4(0, 0, 0, 0);
    const uint32_t r2 = have ? rec_of(g, s2, rep_first) : 0u;
    if (have && XG_BOUND(r2, g.n_states, kBoundState)) rec = *reinterpret_cast<const uint4*>(&g.state[r2]);
    int n_wait = (int)(rec.w & 0xFFFFu);
    if (!XG_BOUND((int)rec.z + n_wait, g.n_wait_edges + 1, kBoundWaitEdge)) n_wait = 0;
    const int incl = warp_inclusive_scan(n_wait, lane);
    const int total = __shfl_sync(kFullWarp, incl, 31);
    for (int p0 = 0; p0 < total; p0 += 32) {
      const int p = p0 + lane;
      const int own = min(owner_of_pair(incl, p, n_here), 31);
      const int first = __shfl_sync(kFullWarp, incl - n_wait, own), wb = __shfl_sync(kFullWarp, (int)rec.z, own);
      const int32_t o2_own = __shfl_sync(kFullWarp, o2, own);
      const uint32_t s2_own = __shfl_sync(kFullWarp, s2, own);
      uint2 we = make_uint2(0xFFFFFFFFu, 0u);
      if (p < total) we = g.wait_edge[wb + (p - first)];
      uint32_t hits = __ballot_sync(kFullWarp, p < total && we.x == rule);
      while (hits) {
        const int h = __ffs(hits) - 1;
        hits &= hits - 1;
        const uint32_t ns = __shfl_sync(kFullWarp, next_word(g, s2_own, we.y), h);
        const int32_t no = __shfl_sync(kFullWarp, (we.y & kSelf) ? o : o2_own, h);
        if (!warp_add_item(st, org, start, cnt, cap, ns, no, lane)) return false;
      }
    }
  }
  return true;
}

template <typename LsbT, typename G>
__device__ __forceinline__ int warp_token_walk(const G& g, const Chart& c, const uint8_t* __restrict__ bytes, int len,
                                               uint32_t* st, int32_t* org, int cap, LsbT* lsb, int* flags, int lane) {
  int cnt = 0;
  const uint32_t rep_first = (uint32_t)g.rep_first;
  const uint32_t* cur_st = c.i_st;
  const int32_t* cur_org = c.i_org;
  int cur_b = 0, cur_e = c.i_cnt;
  if (lane == 0) { lsb[0] = 0; lsb[1] = 0; }
  for (int k = 0; k < len; ++k) {
    const uint32_t byte = bytes[k];
    const uint32_t word = byte >> 5, bit = 1u << (byte & 31);
    const int start = cnt;
    const int self_idx = c.i_idx + k;
    // scan: one (item, edge) pair per lane
    for (int base = cur_b; base < cur_e; base += 32) {
      const int n_here = min(32, cur_e - base);
      const bool have = lane < n_here;
      const uint32_t s = have ? cur_st[base + lane] : 0u;
      const int32_t o = have ? cur_org[base + lane] : 0;
      uint4 ra = make_uint4(0, 0, 0, 0), rb = ra;
      const uint32_t sr = have ? rec_of(g, s, rep_first) : 0u;
      if (have && XG_BOUND(sr, g.n_states, kBoundState)) {
        ra = *reinterpret_cast<const uint4*>(&g.state[sr]);
        rb = *(reinterpret_cast<const uint4*>(&g.state[sr]) + 1);
      }
      int n_edges = (int)(ra.y >> 16);
      if (!XG_BOUND((int)ra.x + n_edges, g.n_scan_edges + 1, kBoundScanEdge)) n_edges = 0;
      const int incl = warp_inclusive_scan(n_edges, lane);
      const int total = __shfl_sync(kFullWarp, incl, 31);
      for (int p0 = 0; p0 < total; p0 += 32) {
        const int p = p0 + lane;
        const int own = min(owner_of_pair(incl, p, n_here), 31);
        const int first = __shfl_sync(kFullWarp, incl - n_edges, own), sb = __shfl_sync(kFullWarp, (int)ra.x, own);
        const int32_t o_own = __shfl_sync(kFullWarp, o, own);
        const uint32_t s_own = __shfl_sync(kFullWarp, s, own);
        const uint32_t e0c = __shfl_sync(kFullWarp, rb.z, own), e0t = __shfl_sync(kFullWarp, rb.w, own);
        uint2 se = make_uint2(kLiteral | 0x100u, 0u);
        if (p < total) se = p == first ? make_uint2(e0c, e0t) : g.scan_edge[sb + (p - first)];      // the first edge is inline in the record
        // the record of the edge's target is requested before the byte is tested against the edge's class: if the edge
        // is taken, the new item's `info` word (and the scan of the next byte) find it on its way
        if (p < total && (se.y & kTarget) < rep_first && XG_BOUND(se.y & kTarget, g.n_states, kBoundState)) asm volatile("prefetch.global.L1 [%0];" ::"l"(&g.state[se.y & kTarget]));
        bool hit = false;
        if (se.x & kLiteral) hit = (se.x & 0x1FFu) == byte;
        else if (XG_BOUND(se.x, g.n_classes, kBoundClass)) hit = (g.class_bits[se.x * 8 + word] & bit) != 0;
        uint32_t hits = __ballot_sync(kFullWarp, hit);
        while (hits) {
          const int h = __ffs(hits) - 1;
          hits &= hits - 1;
          const uint32_t ns = __shfl_sync(kFullWarp, next_word(g, s_own, se.y), h);
          const int32_t no = __shfl_sync(kFullWarp, (se.y & kSelf) ? self_idx : o_own, h);
          if (!warp_add_item(st, org, start, cnt, cap, ns, no, lane)) { *flags |= kWalkOverflow; return k; }
        }
      }
    }
    if (cnt == start) return k;
    // complete (cascades through the growing set): the `info` words of the new items one per lane, then one completion at a time
    for (int q = start; q < cnt;) {
      const int n_here = min(32, cnt - q);
      uint32_t info = 0;
      int32_t o = 0;
      if (lane < n_here) { const uint32_t qr = rec_of(g, st[q + lane], rep_first); if (XG_BOUND(qr, g.n_states, kBoundState)) { info = g.state[qr].info; o = org[q + lane]; } }
      uint32_t done = __ballot_sync(kFullWarp, (info >> 31) != 0);
      q += n_here;
      while (done) {
        const int h = __ffs(done) - 1;
        done &= done - 1;
        const uint32_t rule = __shfl_sync(kFullWarp, info, h) & 0x7FFFFFFFu;
        const int32_t oo = __shfl_sync(kFullWarp, o, h);
        if (oo < 0) continue;             // (an item of unknown context: cache build only, never in a request's chart)
        if (!warp_advance_waiters(g, c, rule, oo, st, org, lsb, start, cnt, cap, lane)) { *flags |= kWalkOverflow; return k; }
      }
    }
    cur_st = st; cur_org = org; cur_b = start; cur_e = cnt;
    if (lane == 0) lsb[k + 2] = (LsbT)cnt;
    __syncwarp();
  }
  return len;
}

// Accept one sampled token of one request (Section 2.2 "trace the output"), by one warp.  The warp
// walks the token's bytes into its scratch (w_st, w_org: kFastCap items, lsb: kFastMaxBytes
// + 2); if every byte survived, the warp appends the new sets behind the request's history, lane
// 0 commits the counters and the warp builds the plan of the next mask.  A rejected token leaves
// the matcher as it was.  With restart_on_eos an accepted end-of-sequence token puts the matcher
// back into its initial state instead of terminating it.  Returns the status, the same in every lane.
template <typename G>
__device__ __forceinline__ int accept_one(MatcherDev& m, const G& g, const VocabDev& v, int tok, bool restart_on_eos, int lane,
                                          uint32_t* w_st, int32_t* w_org, int16_t* lsb) {
  int st = 0;   // XG_OK
  // The token's bytes and the request's current set are each a few dependent loads away (id -> rank -> offset ->
  // bytes; counters -> set bounds -> first item -> its state record).  Both chains are requested before anything is
  // tested, so that they travel together instead of one after the other.
  const bool tok_ok = tok >= 0 && tok < v.vocab_size;
  const int rank = v.id_to_rank[tok_ok ? tok : 0];
  if (!XG_BOUND(rank, v.vocab_size, kBoundTokenRank)) return -6;
  int n_sets = m.n_sets, n_items = m.n_items;
  const Chart c0 = chart_of_history(m.item_state, m.item_origin, m.set_begin, n_sets - 1);
  const uint32_t off = v.offset[rank];
  const int len = (int)(v.offset[rank + 1] - off);
  if (!XG_BOUND((long long)off + len, (long long)v.n_bytes + 1, kBoundTokenBytes)) return -6;
  const bool never = v.never[rank] != 0;
  if (c0.i_cnt > 0 && c0.i_st[0] < (uint32_t)g.rep_first) asm volatile("prefetch.global.L1 [%0];" ::"l"(&g.state[c0.i_st[0]]));
  if (m.terminated) return -8;
  if (!tok_ok) return -7;
  if (tok == v.eos_id) {
    if (lane == 0) {
      if (!root_complete(m, g)) st = -7;
      else if (restart_on_eos) matcher_restart(m, g);
      else m.terminated = 1;
    }
    st = __shfl_sync(0xFFFFFFFFu, st, 0);
    if (st == 0 && restart_on_eos) { __syncwarp(); prepare_plan(m, g, lane); }
    return st;
  }
  if (never || len == 0) return -7;
  int done = 0;
  while (done < len && st == 0) {            // long tokens go through in pieces
    const int piece = min(len - done, kFastMaxBytes);
    int made = 0, slow = 0;
    if (n_sets + piece > m.cap_sets) st = -6;
    else {
      int flags = 0;
      const Chart c = done == 0 ? c0 : chart_of_history(m.item_state, m.item_origin, m.set_begin, n_sets - 1);
      int consumed = warp_token_walk<int16_t>(g, c, v.bytes + off + done, piece, w_st, w_org, kFastCap, lsb, &flags, lane);
      if (flags & kWalkOverflow) {       // the sets do not fit the warp's scratch: the same walk again, exactly, in the matcher's large one
        flags = 0;
        slow = 1;
        consumed = warp_token_walk<int32_t>(g, c, v.bytes + off + done, piece, m.slow_st, m.slow_org, kSlowCap, m.slow_lsb, &flags, lane);
      }
      __syncwarp();
      if (flags & kWalkOverflow) st = -6;
      else if (consumed < piece) st = -7;
      else { made = slow ? m.slow_lsb[piece + 1] : lsb[piece + 1]; if (n_items + made > m.cap_items) st = -6; }
    }
    if (st != 0) break;
    __syncwarp();
    // origins written by the walk are already chart indices (its base is set n_sets - 1);
    // append the new sets behind the history (visible to the next piece; committed below)
    const uint32_t* src_st = slow ? m.slow_st : w_st;
    const int32_t* src_org = slow ? m.slow_org : w_org;
    if (!XG_BOUND(n_items + made, m.cap_items + 1, kBoundChartItem) || !XG_BOUND(n_sets + piece, m.cap_sets + 1, kBoundChartSet)) { st = -6; break; }
    for (int q = lane; q < made; q += 32) { m.item_state[n_items + q] = src_st[q]; m.item_origin[n_items + q] = src_org[q]; }
    for (int j = 1 + lane; j <= piece; j += 32) m.set_begin[n_sets + j] = n_items + (slow ? m.slow_lsb[j + 1] : (int)lsb[j + 1]);
    __syncwarp();
    n_items += made;
    n_sets += piece;
    done += piece;
  }
  if (st == 0) {
    if (lane == 0) { m.n_sets = n_sets; m.n_items = n_items; }
    __syncwarp();
    prepare_plan(m, g, lane);      // the next mask's plan, while the new set is still hot
  }
  return st;
}

// One warp per request: requests follow unrelated paths, so sharing a warp between them would
// serialise their walks.
// kCounts: some grammar of the batch has counted repetitions (otherwise the decoding of state words compiles away)
template <bool kCounts>
__global__ void __launch_bounds__(128)
accept_kernel(MatcherDev* const* __restrict__ matchers, int batch, VocabDev v,
              const int32_t* __restrict__ token_ids, int32_t* __restrict__ status, int restart_on_eos) {
  step_kernel_prologue();
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= batch) return;
  MatcherDev& m = *matchers[b];
  __shared__ uint32_t sh_st[4][kFastCap];
  __shared__ int32_t sh_org[4][kFastCap];
  __shared__ int16_t sh_lsb[4][kFastMaxBytes + 2];
  const int st = accept_one(m, grammar_as<kCounts>(*m.grammar), v, token_ids[b], restart_on_eos != 0, lane, sh_st[threadIdx.x >> 5], sh_org[threadIdx.x >> 5], sh_lsb[threadIdx.x >> 5]);
  if (status && lane == 0) status[b] = st;
}

// ------------------------------------------------------------------------------------------
// Per-step mask, part 1: merge the accepted sets of the current scannable states (run-time
// paragraph of the appendix on the adaptive token mask cache).  grid = (chunks, batch): each
// block owns a slice of one request's row in shared memory, ORs every entry's accepted tokens
// into it (bitsets streamed with coalesced loads, sorted lists cut to the slice by binary
// search) and writes the slice once.
// ------------------------------------------------------------------------------------------
// First index whose element is >= key, in a sorted list.  Called by whole warps with the same
// arguments: 32 probes per round, so a list of a few thousand ids takes three rounds of
// independent loads where a binary search would chain a dozen dependent ones.
__device__ __forceinline__ int lower_bound_u32(const uint32_t* __restrict__ a, int n, uint32_t key) {
  const int lane = threadIdx.x & 31;
  int lo = 0, hi = n;                       // the answer lies in [lo, hi]
  while (lo < hi) {
    const int step = (hi - lo + 31) >> 5;
    const int pos = lo + (lane + 1) * step - 1;                      // ascending with the lane
    const bool less = pos < hi && a[pos] < key;
    const int below = __popc(__ballot_sync(0xFFFFFFFFu, less));      // the probes below the key are the first `below` lanes
    const int first_not_less = lo + (below + 1) * step - 1;          // the probe of lane `below`, if it exists
    lo += below * step;
    hi = first_not_less < hi ? first_not_less : hi;
  }
  return lo;
}

// Visit the ids of a sorted list that fall into [id_lo, id_hi), all threads of the block together.  A short list
// is simply read in full by every block of the cluster (one round of independent loads, no search at all); a
// long one is cut to the slice first.
constexpr int kScanWholeList = 1024;
template <typename F>
__device__ __forceinline__ void for_ids_in_slice(const uint32_t* __restrict__ list, int n, uint32_t id_lo, uint32_t id_hi, F visit) {
  if (n <= kScanWholeList) {
    for (int i = threadIdx.x; i < n; i += blockDim.x) { const uint32_t id = list[i]; if (id >= id_lo && id < id_hi) visit(id); }
  } else {
    const int lo = lower_bound_u32(list, n, id_lo), hi = lo + lower_bound_u32(list + lo, n - lo, id_hi);
    for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) visit(list[i]);
  }
}

// Just-in-time grammars (Section 3.5): while an entry of the current set is not built, the mask
// is the plain definition -- every token walked against the full Earley state.  The bytes the
// current set can scan at all (OR of the per-state first-byte sets) reject most tokens before a
// walk starts.  One warp computes it.
template <typename G>
__device__ __forceinline__ void current_first_bytes(const G& g, const Chart& hist, uint32_t* out8, int lane) {
  if (lane < 8) {
    uint32_t w = 0;
    for (int i = 0; i < hist.i_cnt; ++i) w |= g.state_first[(size_t)rec_of(g, hist.i_st[i]) * 8 + lane];
    out8[lane] = w;
  }
}

// report the plan's missing entries to the host (one thread per request and step)
__device__ __forceinline__ void report_missing(const GrammarDev& g, const StepPlan& plan) {
  JitRing* ring = g.miss_ring;
  if (!ring) return;
  const int n = min(plan.n_missing, kPlanMissingMax);
  for (int z = 0; z < n; ++z) {
    const uint32_t slot = atomicAdd(&ring->count, 1u);
    ring->miss[slot % kJitRingCap] = make_int2(g.jit_slot, plan.missing_state[z]);
  }
}

constexpr int kMergeMaxChunkWords = 2048;

// A token whose walk does not fit the per-thread arrays (more than kFastCap items, or longer than kFastMaxBytes)
// is queued on its request for the exact slow walk; false when the queue is full (the request then fails).
__device__ __forceinline__ bool queue_slow_walk(MatcherDev* m, int token_rank) {
  const int slot = atomicAdd(&m->slow_n, 1);
  if (slot >= kSlowQueue) return false;
  m->slow_q[slot] = token_rank;
  return true;
}

// The queued tokens, one after the other, by one thread: each walked in full from the request's current set (the
// plain definition) in the matcher's large scratch; allow(id) records a token that passes.  false: a walk exceeded
// even that scratch, or the queue had overflowed.
template <typename F, typename G>
__device__ __forceinline__ bool run_slow_walks(MatcherDev* m, const G& g, const VocabDev& v, const Chart& hist, F allow) {
  const int n = m->slow_n;
  if (n > kSlowQueue) return false;
  for (int i = 0; i < n; ++i) {
    const int trank = m->slow_q[i];
    const uint32_t off = v.offset[trank];
    const int len = (int)(v.offset[trank + 1] - off);
    int flags = 0;
    const bool pass = token_walk<int32_t>(g, g.class_bits, hist, v.bytes + off, len, false, m->slow_st, m->slow_org, kSlowCap, m->slow_lsb, &flags, nullptr) == len;
    if (flags & kWalkOverflow) return false;
    if (pass) allow(v.rank_to_id[trank]);
  }
  return true;
}

__global__ void __launch_bounds__(256)
merge_kernel(MatcherDev* const* __restrict__ matchers, VocabDev v, int32_t* __restrict__ bitmask, long long row_stride,
             int32_t* __restrict__ status_user, int32_t* __restrict__ status, int32_t* __restrict__ done_count) {
  __shared__ uint32_t row[kMergeMaxChunkWords];
  __shared__ uint32_t tmp[kMergeMaxChunkWords];
  const int b = blockIdx.y;
  const MatcherDev& m = *matchers[b];
  const GrammarDev& g = *m.grammar;
  const int chunk = (v.n_words + gridDim.x - 1) / gridDim.x;
  const int w0 = blockIdx.x * chunk, w1 = min(v.n_words, w0 + chunk);
  const int nw = max(0, w1 - w0);
  for (int w = threadIdx.x; w < nw; w += blockDim.x) row[w] = 0;
  const StepPlan& plan = *m.plan;
  const int st0 = m.terminated ? -8 : 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    status[b] = st0;
    if (status_user) status_user[b] = st0;
    done_count[b] = 0;
    matchers[b]->slow_n = 0;
  }
  __syncthreads();
  if (st0 == 0 && nw > 0) {
    const uint32_t id_lo = (uint32_t)w0 * 32u, id_hi = (uint32_t)w1 * 32u;
    const int n_merge = plan.n_merge;
    for (int k = 0; k < n_merge; ++k) {
      const EntryDev e = g.entries[plan.merge_state[k]];
      if (e.kind == 2) {
        for (int w = threadIdx.x; w < nw; w += blockDim.x) row[w] |= e.data[w0 + w];
      } else if (e.kind == 0) {
        const int lo = lower_bound_u32(e.data, e.n_list, id_lo), hi = lower_bound_u32(e.data, e.n_list, id_hi);
        for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) { const uint32_t id = e.data[i]; atomicOr(&row[(id >> 5) - w0], 1u << (id & 31)); }
      } else {
        // accepted = everything except the rejected and the uncertain tokens
        const uint32_t tail = (v.vocab_size & 31) ? ((1u << (v.vocab_size & 31)) - 1) : 0xFFFFFFFFu;
        for (int w = threadIdx.x; w < nw; w += blockDim.x) tmp[w] = (w0 + w == v.n_words - 1) ? tail : 0xFFFFFFFFu;
        __syncthreads();
        int lo = lower_bound_u32(e.data, e.n_list, id_lo), hi = lower_bound_u32(e.data, e.n_list, id_hi);
        for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) { const uint32_t id = e.data[i]; atomicAnd(&tmp[(id >> 5) - w0], ~(1u << (id & 31))); }
        lo = lower_bound_u32(e.unc_id, e.n_unc, id_lo); hi = lower_bound_u32(e.unc_id, e.n_unc, id_hi);
        for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) { const uint32_t id = e.unc_id[i]; atomicAnd(&tmp[(id >> 5) - w0], ~(1u << (id & 31))); }
        __syncthreads();
        for (int w = threadIdx.x; w < nw; w += blockDim.x) row[w] |= tmp[w];
      }
      __syncthreads();
    }
    if (threadIdx.x == 0 && v.eos_id >= 0 && (uint32_t)v.eos_id >= id_lo && (uint32_t)v.eos_id < id_hi && plan.eos_ok)
      row[(v.eos_id >> 5) - w0] |= 1u << (v.eos_id & 31);
    __syncthreads();
  }
  for (int w = threadIdx.x; w < nw; w += blockDim.x) bitmask[(long long)b * row_stride + w0 + w] = (int32_t)row[w];
}

// ------------------------------------------------------------------------------------------
// Per-step mask, part 2: check the uncertain tokens of the current scannable states against
// the request's full Earley state (Section 3.4).  grid = (slices, batch).
//
// An uncertain token of entry (state q, origin o) fails inside q's rule; its only way to be
// allowed is to leave the rule at one of its recorded exit offsets and continue in the context.
// What the context looks like right after the rule completes does not depend on the token: it
// is the set obtained by completing rule(q) started at o.  That continuation set is computed
// once per entry, together with the set of bytes it can scan; each token then needs one bit
// test per exit, and only the survivors walk their remaining bytes from the continuation set.
// Tokens are taken in trie order, one per lane, so neighbouring lanes share prefixes.
// The last block of a request to finish clears the row if anything overflowed.
// ------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(256)
check_kernel(MatcherDev* const* __restrict__ matchers, VocabDev v, int32_t* __restrict__ bitmask, long long row_stride,
             int32_t* __restrict__ status_user, int32_t* __restrict__ status, int32_t* __restrict__ done_count) {
  __shared__ const uint32_t* ent_rank[kPlanCheckMax];
  __shared__ const uint32_t* ent_exit[kPlanCheckMax];
  __shared__ int ent_cum[kPlanCheckMax + 1];
  __shared__ uint32_t cont_st[kPlanCheckMax][kContCap];
  __shared__ int32_t cont_org[kPlanCheckMax][kContCap];
  __shared__ int cont_cnt[kPlanCheckMax];
  __shared__ uint32_t cont_first[kPlanCheckMax][8];
  __shared__ uint32_t sh_class[kSharedClasses * 8];
  __shared__ int sh_fail;
  __shared__ int sh_last;
  const int b = blockIdx.y;
  const MatcherDev& m = *matchers[b];
  const GrammarDev& g = *m.grammar;
  const StepPlan& plan = *m.plan;
  const int n = m.n_sets - 1;
  MatcherDev* mw = matchers[b];
  const bool live = !m.terminated;
  // an entry is not built yet, or the plan did not fit its fixed arrays: walk the whole vocabulary instead
  const bool fallback = live && (plan.n_missing > 0 || plan.overflow);
  const int n_ent = (live && !fallback) ? plan.n_check : 0;
  const int total = n_ent ? plan.check_cum[n_ent] : 0;
  const int stride = gridDim.x * blockDim.x;
  if (threadIdx.x == 0) sh_fail = 0;
  if (fallback) {
    __shared__ uint32_t set_first[8];
    const Chart hist = chart_of_history(m.item_state, m.item_origin, m.set_begin, n);
    const uint32_t* class_bits = stage_class_bits(g, sh_class);
    current_first_bytes(g, hist, set_first, threadIdx.x);
    if (blockIdx.x == 0 && threadIdx.x == 0 && plan.n_missing > 0) report_missing(g, plan);
    __syncthreads();
    uint32_t* row = (uint32_t*)bitmask + (long long)b * row_stride;
    for (int r = blockIdx.x * blockDim.x + threadIdx.x; r < v.vocab_size; r += stride) {
      if (v.never[r]) continue;
      const uint32_t off = v.offset[r];
      const int len = (int)(v.offset[r + 1] - off);
      const uint32_t byte = v.bytes[off];
      if (!((set_first[byte >> 5] >> (byte & 31)) & 1u)) continue;
      if (len > kFastMaxBytes) { if (!queue_slow_walk(mw, r)) sh_fail = 1; continue; }
      uint32_t st[kFastCap];
      int32_t org[kFastCap];
      int16_t lsb[kFastMaxBytes + 2];
      int flags = 0;
      const bool pass = token_walk<int16_t>(g, class_bits, hist, v.bytes + off, len, false, st, org, kFastCap, lsb, &flags, nullptr) == len;
      if (flags & kWalkOverflow) { if (!queue_slow_walk(mw, r)) sh_fail = 1; }
      else if (pass) { const int id = v.rank_to_id[r]; atomicOr(&row[id >> 5], 1u << (id & 31)); }
    }
  } else
  if (blockIdx.x * (int)blockDim.x < total) {         // blocks without candidates only take part in the count below
    const Chart hist = chart_of_history(m.item_state, m.item_origin, m.set_begin, n);
    const uint32_t* class_bits = stage_class_bits(g, sh_class);
    // the plan's arrays for the live entries, copied with coalesced loads
    for (int i = threadIdx.x; i < n_ent; i += blockDim.x) {
      const EntryDev& e = g.entries[plan.check_state[i]];
      ent_rank[i] = e.chk_rank; ent_exit[i] = e.chk_exit;
      cont_cnt[i] = plan.cont_cnt[i];
    }
    for (int i = threadIdx.x; i <= n_ent; i += blockDim.x) ent_cum[i] = plan.check_cum[i];
    for (int i = threadIdx.x; i < n_ent * kContCap; i += blockDim.x) {
      (&cont_st[0][0])[i] = (&plan.cont_st[0][0])[i];
      (&cont_org[0][0])[i] = (&plan.cont_org[0][0])[i];
    }
    for (int i = threadIdx.x; i < n_ent * 8; i += blockDim.x) (&cont_first[0][0])[i] = (&plan.cont_first[0][0])[i];
    __syncthreads();
    uint32_t* row = (uint32_t*)bitmask + (long long)b * row_stride;
  constexpr int kUnroll = 4;
  for (int j0 = blockIdx.x * blockDim.x + threadIdx.x; j0 < total; j0 += kUnroll * stride) {
    // filter phase: four candidates per thread with their loads in flight together; nearly all
    // of them end here, on the first-byte test of their (usually single) exit
    int ent[kUnroll], rank[kUnroll];
    uint32_t exits[kUnroll], off[kUnroll], nxt[kUnroll], byte0[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int j = j0 + u * stride;
      rank[u] = -1;
      exits[u] = 0;
      if (j < total) {
        int e = 0;
        while (j >= ent_cum[e + 1]) ++e;
        ent[u] = e;
        rank[u] = (int)ent_rank[e][j - ent_cum[e]];
        exits[u] = ent_exit[e][j - ent_cum[e]];
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      if (rank[u] >= 0) { off[u] = v.offset[rank[u]]; nxt[u] = v.offset[rank[u] + 1]; }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      if (rank[u] >= 0 && exits[u]) byte0[u] = v.bytes[off[u] + __ffs(exits[u]) - 1];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      if (rank[u] < 0) continue;
      const int e = ent[u];
      const int len = (int)(nxt[u] - off[u]);
      bool pass = false, overflow = false;
      if (exits[u] == 0) {
        // no exit record (very long token, or its walk overflowed at build time): walk in full
        if (len > kFastMaxBytes) overflow = true;      // (queued for the slow walk below)
        else {
          uint32_t st[kFastCap];
          int32_t org[kFastCap];
          int16_t lsb[kFastMaxBytes + 2];
          int flags = 0;
          pass = token_walk<int16_t>(g, class_bits, hist, v.bytes + off[u], len, false, st, org, kFastCap, lsb, &flags, nullptr) == len;
          overflow = (flags & kWalkOverflow) != 0;
        }
      } else {
        uint32_t left = exits[u];
        bool first = true;
        while (left && !pass && !overflow) {
          const int at = __ffs(left) - 1;
          left &= left - 1;
          const uint32_t byte = first ? byte0[u] : v.bytes[off[u] + at];
          first = false;
          if (!((cont_first[e][byte >> 5] >> (byte & 31)) & 1u)) continue;
          uint32_t st[kFastCap];
          int32_t org[kFastCap];
          int16_t lsb[kFastMaxBytes + 2];
          int flags = 0;
          Chart c = hist;
          c.i_st = cont_st[e]; c.i_org = cont_org[e]; c.i_cnt = cont_cnt[e]; c.i_idx = n + at;
          pass = token_walk<int16_t>(g, class_bits, c, v.bytes + off[u] + at, len - at, false, st, org, kFastCap, lsb, &flags, nullptr) == len - at;
          overflow = (flags & kWalkOverflow) != 0;
        }
      }
      if (overflow) { if (!queue_slow_walk(mw, rank[u])) sh_fail = 1; }       // the whole token again, exactly
      else if (pass) { const int id = v.rank_to_id[rank[u]]; atomicOr(&row[id >> 5], 1u << (id & 31)); }
    }
  }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (sh_fail) atomicExch(&status[b], -6);
    __threadfence();
    sh_last = atomicAdd(&done_count[b], 1) == (int)gridDim.x - 1;
  }
  __syncthreads();
  if (sh_last) {
    __threadfence();
    // every block of the request has finished: the queued slow walks, by one thread
    if (threadIdx.x == 0 && *(volatile int32_t*)&mw->slow_n > 0) {
      uint32_t* row = (uint32_t*)bitmask + (long long)b * row_stride;
      const Chart hist = chart_of_history(m.item_state, m.item_origin, m.set_begin, n);
      if (!run_slow_walks(mw, g, v, hist, [&](int id) { row[id >> 5] |= 1u << (id & 31); })) status[b] = -6;
      __threadfence();
    }
    __syncthreads();
    const int s = *(volatile int32_t*)&status[b];
    if (s == -6) {
      uint32_t* row = (uint32_t*)bitmask + (long long)b * row_stride;
      for (int w = threadIdx.x; w < v.n_words; w += blockDim.x) row[w] = 0;
      if (threadIdx.x == 0 && status_user) status_user[b] = -6;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Mask apply (Section 2.1): logits of disallowed tokens become -inf, in place, one pass.
// One 16-byte vector per thread and step.  A vector whose tokens are all allowed is skipped
// (neither read nor written); one whose tokens are all disallowed is overwritten without being
// read; only mixed vectors are read, blended and written back.
// ------------------------------------------------------------------------------------------
template <int ELEMS>
__device__ __forceinline__ uint4 blend_ninf(uint4 x, uint32_t bits) {
  if (ELEMS == 8) {
    // four allowed-bits -> four bytes of 0x00 / 0xFF (a multiply spreads the bits to the bytes' low bits, a second
    // one fills the bytes), then each byte is doubled into the 16-bit lane it stands for
    const uint32_t lo = (((bits & 0xFu) * 0x00204081u) & 0x01010101u) * 0xFFu;
    const uint32_t hi = ((((bits >> 4) & 0xFu) * 0x00204081u) & 0x01010101u) * 0xFFu;
    const uint32_t k0 = __byte_perm(lo, 0u, 0x1100), k1 = __byte_perm(lo, 0u, 0x3322);
    const uint32_t k2 = __byte_perm(hi, 0u, 0x1100), k3 = __byte_perm(hi, 0u, 0x3322);
    constexpr uint32_t kNinf2 = 0xFF80FF80u;
    return make_uint4((x.x & k0) | (kNinf2 & ~k0), (x.y & k1) | (kNinf2 & ~k1), (x.z & k2) | (kNinf2 & ~k2), (x.w & k3) | (kNinf2 & ~k3));
  }
  if (!(bits & 1u)) x.x = 0xFF800000u;
  if (!(bits & 2u)) x.y = 0xFF800000u;
  if (!(bits & 4u)) x.z = 0xFF800000u;
  if (!(bits & 8u)) x.w = 0xFF800000u;
  return x;
}

// The vectors [v_begin, v_end) of one row, by `n_threads` threads of which this is thread `tid`; word_at(w) gives
// word w of the row's mask.  Each thread handles four vectors per iteration: the four mask tests first, then the
// loads of the mixed vectors (independent, all in flight together), then the stores.
template <int ELEMS, typename MaskFn>   // elements per 16-byte vector: 8 (bf16) or 4 (fp32)
__device__ __forceinline__ void apply_vectors(uint4* __restrict__ base, int v_begin, int v_end, int tid, int n_threads, MaskFn word_at) {
  constexpr uint32_t kAll = (1u << ELEMS) - 1;
  const uint4 ninf = ELEMS == 8 ? make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u)
                                : make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u);
  for (int v0 = v_begin + tid; v0 < v_end; v0 += 4 * n_threads) {
    uint32_t bits[4];
    uint4 x[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int vi = v0 + u * n_threads;
      const int first = vi * ELEMS;
      bits[u] = vi < v_end ? ((word_at(first >> 5) >> (first & 31)) & kAll) : kAll;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (bits[u] != kAll && bits[u] != 0) x[u] = __ldcs(&base[v0 + u * n_threads]);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (bits[u] == kAll) continue;
      __stcs(&base[v0 + u * n_threads], bits[u] == 0 ? ninf : blend_ninf<ELEMS>(x[u], bits[u]));
    }
  }
}

// the elements behind a row's last whole vector (vocab_size not a multiple of the vector width)
template <int ELEMS, typename MaskFn>
__device__ __forceinline__ void apply_ragged_tail(void* row_base, int vocab_size, int tid, int n_threads, MaskFn word_at) {
  for (int c = (vocab_size / ELEMS) * ELEMS + tid; c < vocab_size; c += n_threads) {
    if ((word_at(c >> 5) >> (c & 31)) & 1u) continue;
    if (ELEMS == 8) ((uint16_t*)row_base)[c] = 0xFF80u;
    else ((uint32_t*)row_base)[c] = 0xFF800000u;
  }
}

// grid = (blocks per row, rows)
template <int ELEMS>
__global__ void __launch_bounds__(256)
apply_kernel(void* __restrict__ logits, int vocab_size, long long row_stride_elems, const uint32_t* __restrict__ bitmask,
             long long mask_stride, const int32_t* __restrict__ row_indices) {
  step_kernel_prologue();
  const int r = row_indices ? row_indices[blockIdx.y] : blockIdx.y;
  const uint32_t* mrow = bitmask + (long long)r * mask_stride;
  void* row_base = ELEMS == 8 ? (void*)((uint16_t*)logits + (long long)r * row_stride_elems) : (void*)((uint32_t*)logits + (long long)r * row_stride_elems);
  auto word_at = [&](int w) { return __ldg(&mrow[w]); };
  apply_vectors<ELEMS>((uint4*)row_base, 0, vocab_size / ELEMS, blockIdx.x * blockDim.x + threadIdx.x, gridDim.x * blockDim.x, word_at);
  if (blockIdx.x == 0) apply_ragged_tail<ELEMS>(row_base, vocab_size, threadIdx.x, blockDim.x, word_at);
}

// ------------------------------------------------------------------------------------------
// Per-step mask in one launch: a thread-block cluster of two to eight blocks per request.  Block
// r of the cluster keeps slice r of the request's row in its shared memory.
//   1. every block merges the accepted sets of the plan's entries into its own slice;
//   2. cluster barrier; the blocks share the uncertain candidates (trie order, one token per
//      lane); a token that passes is OR-ed into the slice of the block that owns its id, through
//      distributed shared memory;
//   3. cluster barrier; every block writes its slice with coalesced stores.
// No global atomics, no scratch words, and the row never makes a round trip through L2.
// With kAccept the launch first accepts one sampled token per request (the first warp of the
// cluster's block 0, as in accept_kernel; the rest of the cluster waits at a cluster barrier) and
// then fills the mask of the state it reached: in a decode loop the two always follow each other,
// and one launch saves a kernel boundary and lets a request with a slow accept and a short fill
// overlap one with the opposite mix.
// With kApplyElems (8: bf16 logits, 4: fp32) each block also masks its slice of the request's logits row from
// the slice it has just written, still in shared memory: the mask is not read back from global memory, there is
// no kernel boundary between fill and apply, and the rows of requests whose fill is short are masked while
// other requests still walk their uncertain tokens.
// The host picks cluster and block size so that the whole batch is resident at once.  Used when
// a slice fits (at most 2048 words per block); larger vocabularies take the two-kernel path above.
// ------------------------------------------------------------------------------------------
constexpr int kMaxClusterBlocks = 8;      // the portable cluster size limit

// launched with a cluster of gridDim.x blocks (2, 4 or 8) along x
// kHeavy: the launch may hold requests with hundreds of uncertain candidates (a grammar of the batch has an entry with
// a long check list); only then does the kernel carry the second-byte sets and the walk queues described below.
// kCounts: some grammar of the batch has counted repetitions (Section 3.6); without, state words need no decoding.
template <bool kAccept, int kApplyElems, bool kHeavy, bool kCounts>
__global__ void __launch_bounds__(256, 4)
fill_cluster_kernel(MatcherDev* const* __restrict__ matchers, VocabDev v, int32_t* __restrict__ bitmask, long long row_stride,
                    int32_t* __restrict__ status_user, const int32_t* __restrict__ token_ids, int32_t* __restrict__ accept_status,
                    int restart_on_eos, void* __restrict__ logits, long long logits_row_stride_elems) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ uint32_t dyn_smem[];          // this block's row slice and a scratch slice: 2 x ceil(W / blocks) words
  __shared__ const uint32_t* ent_rank[kPlanCheckMax];
  __shared__ const uint32_t* ent_exit[kPlanCheckMax];
  __shared__ const uint32_t* ent_info[kPlanCheckMax];
  __shared__ int ent_cum[kPlanCheckMax + 1];
  __shared__ uint32_t cont_st[kPlanCheckMax][kContCap];
  __shared__ int32_t cont_org[kPlanCheckMax][kContCap];
  __shared__ int cont_cnt[kPlanCheckMax];
  __shared__ uint32_t cont_first[kPlanCheckMax][8];
  __shared__ uint32_t sh_class[kSharedClasses * 8];
  // scratch of the accepting warp (kAccept)
  __shared__ uint32_t acc_st[kAccept ? kFastCap : 1];
  __shared__ int32_t acc_org[kAccept ? kFastCap : 1];
  __shared__ int16_t acc_lsb[kAccept ? kFastMaxBytes + 2 : 1];
  __shared__ int sh_fail;          // set in every block of the cluster when any of them fails
  __shared__ int sh_slow;          // set in every block of the cluster when a token was queued for the exact slow walk
  // Second-byte sets.  What a token has left after its exit starts with byte b1, which the entry's continuation set
  // must be able to scan; the set that scan leads to -- and so the bytes b2 it can scan in turn -- depends only
  // on (entry, b1), not on the token.  For requests with many candidates every block works these sets out once,
  // one thread per (entry, b1) pair: a token is then decided by two bit tests when it has at most two bytes left,
  // and most of the others die on their second byte without a walk.
  constexpr int kPairs = kHeavy ? 96 : 1, kPairsMinCandidates = 1024;
  __shared__ __align__(16) uint32_t pair_second[kPairs][8];      // written as two 16-byte vectors per pair
  __shared__ int pair_base[kHeavy ? kPlanCheckMax + 1 : 1];
  __shared__ uint8_t pair_unknown[kPairs];      // the pair's walk did not fit the fast arrays: its tokens are walked
  __shared__ int pair_n;           // pairs built (0: no second-byte sets for this request)
  // Walks that survive both byte tests cluster in a few warps (tokens with a common prefix are neighbours in the
  // candidate lists), and the lanes of a warp walk one after the other wherever their paths differ.  For requests with
  // many candidates the surviving (token, exit) pairs therefore go through queues, one per block of the cluster,
  // filled round robin so that every block gets an equal share of every run, and each block deals its queue out over
  // its warps first and over the lanes of a warp last.
  constexpr int kWalkQueue = kHeavy ? 192 : 1;
  __shared__ uint2 walk_q[kWalkQueue];          // (token rank, entry | exit offset << 8)
  __shared__ int walk_q_n;

  step_kernel_prologue();
  const int b = blockIdx.y;
  const int rank = (int)cluster.block_rank();
  MatcherDev* mw = matchers[b];
  const MatcherDev& m = *matchers[b];
  const typename GrammarAs<kCounts>::type& g = grammar_as<kCounts>(*m.grammar);
  const StepPlan& plan = *m.plan;
  const int n_blocks = (int)gridDim.x;
  const int chunk = (v.n_words + n_blocks - 1) / n_blocks;
  uint32_t* row = dyn_smem;
  uint32_t* tmp = dyn_smem + chunk;
  const int w0 = rank * chunk, w1 = min(v.n_words, w0 + chunk);
  const int nw = max(0, w1 - w0);
  for (int w = threadIdx.x; w < nw; w += blockDim.x) row[w] = 0;
  if (kAccept) {
    // nothing of the request's state or plan is read before this barrier; its release/acquire pair makes what the
    // accepting warp wrote visible to the whole cluster
    if (rank == 0 && threadIdx.x < 32) {
      const int st = accept_one(*matchers[b], g, v, token_ids[b], restart_on_eos != 0, (int)threadIdx.x, acc_st, acc_org, acc_lsb);
      if (accept_status && threadIdx.x == 0) accept_status[b] = st;
    }
    cluster.sync();
  }
  const int st0 = m.terminated ? -8 : 0;
  if (threadIdx.x == 0) { sh_fail = 0; sh_slow = 0; }
  // an entry is not built yet, or the plan did not fit its fixed arrays: walk the whole vocabulary instead
  const bool fallback = st0 == 0 && (plan.n_missing > 0 || plan.overflow);
  const int n_ent = (st0 == 0 && !fallback) ? plan.n_check : 0;
  const int total = n_ent ? plan.check_cum[n_ent] : 0;
  __shared__ uint32_t set_first[8];
  __syncthreads();
  // 1. merge
  if (st0 == 0 && nw > 0) {
    const uint32_t id_lo = (uint32_t)w0 * 32u, id_hi = (uint32_t)w1 * 32u;
    const int n_merge = plan.n_merge;
    for (int k = 0; k < n_merge; ++k) {
      const EntryDev e = g.entries[plan.merge_state[k]];
      if (e.kind == 2) {
        for (int w = threadIdx.x; w < nw; w += blockDim.x) row[w] |= e.data[w0 + w];
      } else if (e.kind == 0) {
        for_ids_in_slice(e.data, e.n_list, id_lo, id_hi, [&](uint32_t id) { atomicOr(&row[(id >> 5) - w0], 1u << (id & 31)); });
      } else {
        const uint32_t tail = (v.vocab_size & 31) ? ((1u << (v.vocab_size & 31)) - 1) : 0xFFFFFFFFu;
        for (int w = threadIdx.x; w < nw; w += blockDim.x) tmp[w] = (w0 + w == v.n_words - 1) ? tail : 0xFFFFFFFFu;
        __syncthreads();
        for_ids_in_slice(e.data, e.n_list, id_lo, id_hi, [&](uint32_t id) { atomicAnd(&tmp[(id >> 5) - w0], ~(1u << (id & 31))); });
        for_ids_in_slice(e.unc_id, e.n_unc, id_lo, id_hi, [&](uint32_t id) { atomicAnd(&tmp[(id >> 5) - w0], ~(1u << (id & 31))); });
        __syncthreads();
        for (int w = threadIdx.x; w < nw; w += blockDim.x) row[w] |= tmp[w];
      }
      __syncthreads();
    }
    if (threadIdx.x == 0 && v.eos_id >= 0 && (uint32_t)v.eos_id >= id_lo && (uint32_t)v.eos_id < id_hi && plan.eos_ok)
      row[(v.eos_id >> 5) - w0] |= 1u << (v.eos_id & 31);
  }
  // 2. check (the plan and its arrays are the same for the whole cluster: `total` and `fallback` are uniform)
  if (total > 0 || fallback) {
    const int n = m.n_sets - 1;
    const Chart hist = chart_of_history(m.item_state, m.item_origin, m.set_begin, n);
    const uint32_t* class_bits = stage_class_bits(g, sh_class);
    for (int i = threadIdx.x; i < n_ent; i += blockDim.x) {
      const EntryDev& e = g.entries[plan.check_state[i]];
      ent_rank[i] = e.chk_rank; ent_exit[i] = e.chk_exit; ent_info[i] = e.chk_info;
      cont_cnt[i] = plan.cont_cnt[i];
    }
    for (int i = threadIdx.x; i <= n_ent; i += blockDim.x) ent_cum[i] = plan.check_cum[i];
    for (int i = threadIdx.x; i < n_ent * kContCap; i += blockDim.x) {
      (&cont_st[0][0])[i] = (&plan.cont_st[0][0])[i];
      (&cont_org[0][0])[i] = (&plan.cont_org[0][0])[i];
    }
    for (int i = threadIdx.x; i < n_ent * 8; i += blockDim.x) (&cont_first[0][0])[i] = (&plan.cont_first[0][0])[i];
    if (fallback) {
      current_first_bytes(g, hist, set_first, threadIdx.x);
      if (rank == 0 && threadIdx.x == 0 && plan.n_missing > 0) report_missing(g, plan);
    }
    if (rank == 0 && threadIdx.x == 0) mw->slow_n = 0;
    if (threadIdx.x == 0) { pair_n = 0; walk_q_n = 0; }
    uint32_t w_st[kFastCap];                       // this thread's walk arrays
    int32_t w_org[kFastCap];
    int16_t w_lsb[kFastMaxBytes + 2];
    if (kHeavy && total >= kPairsMinCandidates) {  // (uniform over the cluster)
      __syncthreads();                             // the staged continuation sets are visible
      if (threadIdx.x == 0) {
        int run = 0;
        for (int e = 0; e < n_ent; ++e) {
          pair_base[e] = run;
          for (int w = 0; w < 8; ++w) run += __popc(cont_first[e][w]);
        }
        pair_base[n_ent] = run;
        pair_n = run <= kPairs ? run : 0;          // too many pairs for the table: no second-byte sets
      }
      __syncthreads();
      for (int p = threadIdx.x; p < pair_n; p += blockDim.x) {
        int e = 0;
        while (p >= pair_base[e + 1]) ++e;
        int skip = p - pair_base[e], b1 = 0;       // b1 = the (skip)-th byte of the entry's first-byte set
        for (int w = 0; w < 8; ++w) {
          uint32_t bits = cont_first[e][w];
          const int c = __popc(bits);
          if (skip >= c) { skip -= c; continue; }
          while (skip--) bits &= bits - 1;
          b1 = 32 * w + __ffs(bits) - 1;
          break;
        }
        int flags = 0;
        const uint8_t one_byte = (uint8_t)b1;
        Chart c = hist;
        c.i_st = cont_st[e]; c.i_org = cont_org[e]; c.i_cnt = cont_cnt[e]; c.i_idx = n + 1;
        const int consumed = token_walk<int16_t>(g, class_bits, c, &one_byte, 1, false, w_st, w_org, kFastCap, w_lsb, &flags, nullptr);
        uint4 fa = make_uint4(0, 0, 0, 0), fb = make_uint4(0, 0, 0, 0);
        const bool unknown = (flags & kWalkOverflow) || consumed != 1;
        pair_unknown[p] = unknown ? 1 : 0;
        if (unknown) fa = fb = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);    // every token goes on to its walk
        else
          for (int q = 0; q < w_lsb[2]; ++q) {
            const uint4* sf = reinterpret_cast<const uint4*>(g.state_first + (size_t)rec_of(g, w_st[q]) * 8);
            const uint4 a = sf[0], d = sf[1];
            fa.x |= a.x; fa.y |= a.y; fa.z |= a.z; fa.w |= a.w;
            fb.x |= d.x; fb.y |= d.y; fb.z |= d.z; fb.w |= d.w;
          }
        uint4* out = reinterpret_cast<uint4*>(pair_second[p]);
        out[0] = fa; out[1] = fb;
      }
    }
    cluster.sync();            // every slice is merged (and this block's staging, and the emptied slow queue, are visible)
    const int stride = n_blocks * blockDim.x;
    // a failure (rare) is recorded in every block's flag, so that each block reads its own at the end and no block has to
    // outlive the others' reads
    auto fail_everywhere = [&]() { for (int r = 0; r < n_blocks; ++r) atomicOr(cluster.map_shared_rank(&sh_fail, r), 1); };
    // a walk that does not fit the per-thread arrays: the token is queued for the exact slow walk after the others
    auto walk_slowly = [&](int trank) {
      if (!queue_slow_walk(mw, trank)) fail_everywhere();
      for (int r = 0; r < n_blocks; ++r) atomicOr(cluster.map_shared_rank(&sh_slow, r), 1);
    };
    auto walk_one = [&](int trank, uint32_t off, int e, int at) {
      const int len = (int)(v.offset[trank + 1] - off);
      bool pass = false, overflow = len - at > kFastMaxBytes;
      if (!overflow) {
        int flags = 0;
        Chart c = hist;
        if (at > 0) { c.i_st = cont_st[e]; c.i_org = cont_org[e]; c.i_cnt = cont_cnt[e]; c.i_idx = n + at; }
        pass = token_walk<int16_t>(g, class_bits, c, v.bytes + off + at, len - at, false, w_st, w_org, kFastCap, w_lsb, &flags, nullptr) == len - at;
        overflow = (flags & kWalkOverflow) != 0;
      }
      if (overflow) walk_slowly(trank);
      return pass && !overflow;
    };
    if (fallback) {
      // the plain definition: every token against the full Earley state, in trie order
      for (int r = rank * blockDim.x + threadIdx.x; r < v.vocab_size; r += stride) {
        if (v.never[r]) continue;
        const uint32_t off = v.offset[r];
        const uint32_t byte = v.bytes[off];
        if (!((set_first[byte >> 5] >> (byte & 31)) & 1u)) continue;
        if ((int)(v.offset[r + 1] - off) > kFastMaxBytes) { walk_slowly(r); continue; }
        if (walk_one(r, off, 0, 0)) {
          const int id = v.rank_to_id[r];
          const int word = id >> 5, owner = word / chunk;
          if (XG_BOUND(word, v.n_words, kBoundRowWord) && XG_BOUND(owner, n_blocks, kBoundClusterBlock))
            atomicOr(cluster.map_shared_rank(&row[word - owner * chunk], owner), 1u << (id & 31));
        }
      }
    }
    const bool queued = kHeavy && total >= kPairsMinCandidates;       // (uniform over the cluster)
    // one candidate whose exit mask, token rank and (for the survivors of the first test) offsets are already here
    auto check_candidate = [&](int j, int e, int trank, uint32_t left, uint32_t off, int len) {
      bool pass = false;
      while (left && !pass) {
        const int at = __ffs(left) - 1;
        left &= left - 1;
        const uint32_t byte = v.bytes[off + at];
        if (!((cont_first[e][byte >> 5] >> (byte & 31)) & 1u)) continue;
        // a single byte left that the continuation set can scan: the set after it is not empty, nothing to walk
        if (at + 1 == len) { pass = true; break; }
        if (kHeavy && pair_n > 0) {
          int p = pair_base[e];
          for (uint32_t w = 0; w < (byte >> 5); ++w) p += __popc(cont_first[e][w]);
          p += __popc(cont_first[e][byte >> 5] & ((1u << (byte & 31)) - 1u));
          const uint32_t b2 = v.bytes[off + at + 1];
          if (!((pair_second[p][b2 >> 5] >> (b2 & 31)) & 1u)) continue;          // dies on its second byte
          if (at + 2 == len && !pair_unknown[p]) { pass = true; break; }
        }
        if (queued) {             // the walk goes to the queue of block (j mod blocks); a full queue: walk here after all
          const int target = j % n_blocks;
          const int slot = atomicAdd(cluster.map_shared_rank(&walk_q_n, target), 1);
          if (slot < kWalkQueue) { *cluster.map_shared_rank(&walk_q[slot], target) = make_uint2((uint32_t)trank, (uint32_t)e | ((uint32_t)at << 8)); continue; }
        }
        pass = walk_one(trank, off, e, at);
      }
      if (pass) {
        const int id = v.rank_to_id[trank];
        const int word = id >> 5, owner = word / chunk;
        if (XG_BOUND(word, v.n_words, kBoundRowWord) && XG_BOUND(owner, n_blocks, kBoundClusterBlock))
          atomicOr(cluster.map_shared_rank(&row[word - owner * chunk], owner), 1u << (id & 31));
      }
    };
    for (int j = rank * blockDim.x + threadIdx.x; j < total; j += stride) {
      // per candidate: its exit mask and the byte at its first exit, both streamed in list order;
      // the token's rank and bytes are only touched by the few that survive the bit test
      int e = 0;
      while (j >= ent_cum[e + 1]) ++e;
      const int k = j - ent_cum[e];
      if (!XG_BOUND(e, n_ent, kBoundPlanEntry) || !XG_BOUND(k, ent_cum[e + 1] - ent_cum[e], kBoundCheckList)) continue;
      uint32_t left = ent_exit[e][k];
      const int trank = (int)ent_rank[e][k];      // read together with the exit mask: one dependent load less for the survivors
      if (!XG_BOUND(trank, v.vocab_size, kBoundTokenRank)) continue;
      if (left == 0) {                // no exit record (very long token, or its build-time walk overflowed): walk in full
        if ((int)(v.offset[trank + 1] - v.offset[trank]) > kFastMaxBytes) { walk_slowly(trank); continue; }
        if (walk_one(trank, v.offset[trank], e, 0)) {
          const int id = v.rank_to_id[trank];
          const int word = id >> 5, owner = word / chunk;
          if (XG_BOUND(word, v.n_words, kBoundRowWord) && XG_BOUND(owner, n_blocks, kBoundClusterBlock))
            atomicOr(cluster.map_shared_rank(&row[word - owner * chunk], owner), 1u << (id & 31));
        }
        continue;
      }
      // The first exit (for most tokens the only one) is decided from the list alone: its byte against the bytes the
      // continuation set can scan, the next byte against the second-byte set of that pair, and with at most two bytes
      // left the token is allowed without a walk.  Only what is still open after that touches the vocabulary tables.
      const uint32_t info = ent_info[e][k];
      const uint32_t b1 = info & 0xFFu, b2 = (info >> 8) & 0xFFu, rem = info >> 16;
      const int at1 = __ffs(left) - 1;
      int first = 0;                                  // the first exit: 0 dead, 1 allowed, 2 has to be walked
      if ((cont_first[e][b1 >> 5] >> (b1 & 31)) & 1u) {
        first = rem == 1 ? 1 : 2;
        if (kHeavy && rem > 1 && pair_n > 0) {
          int p = pair_base[e];
          for (uint32_t w = 0; w < (b1 >> 5); ++w) p += __popc(cont_first[e][w]);
          p += __popc(cont_first[e][b1 >> 5] & ((1u << (b1 & 31)) - 1u));
          if (!((pair_second[p][b2 >> 5] >> (b2 & 31)) & 1u)) first = 0;              // dies on its second byte
          else if (rem == 2 && !pair_unknown[p]) first = 1;
        }
      }
      if (first == 1) {
        const int id = v.rank_to_id[trank];
        const int word = id >> 5, owner = word / chunk;
        if (XG_BOUND(word, v.n_words, kBoundRowWord) && XG_BOUND(owner, n_blocks, kBoundClusterBlock))
          atomicOr(cluster.map_shared_rank(&row[word - owner * chunk], owner), 1u << (id & 31));
        continue;
      }
      if (first == 2 && queued) {                     // its walk goes to the queue of block (j mod blocks)
        const int target = j % n_blocks;
        const int slot = atomicAdd(cluster.map_shared_rank(&walk_q_n, target), 1);
        if (slot < kWalkQueue) { *cluster.map_shared_rank(&walk_q[slot], target) = make_uint2((uint32_t)trank, (uint32_t)e | ((uint32_t)at1 << 8)); first = 0; }
      }
      if (first == 0) left &= left - 1;               // the first exit is settled (dead, or queued); any others go the general way
      if (left == 0) continue;                        // the usual end of a candidate
      const uint32_t off = v.offset[trank];
      check_candidate(j, e, trank, left, off, (int)(v.offset[trank + 1] - off));
    }
    if (queued) {
      cluster.sync();          // every queue is complete
      const int n_q = min(walk_q_n, kWalkQueue), n_warps = (int)(blockDim.x >> 5);
      // entry i goes to warp i mod warps, lane i / warps: a short queue puts one walk into every warp before a second
      const int mine = (int)(threadIdx.x >> 5) + (int)(threadIdx.x & 31) * n_warps;
      for (int i = mine; i < n_q; i += (int)blockDim.x) {
        const uint2 entry = walk_q[i];
        const int trank = (int)entry.x;
        if (walk_one(trank, v.offset[trank], (int)(entry.y & 0xFFu), (int)(entry.y >> 8))) {
          const int id = v.rank_to_id[trank];
          const int word = id >> 5, owner = word / chunk;
          if (XG_BOUND(word, v.n_words, kBoundRowWord) && XG_BOUND(owner, n_blocks, kBoundClusterBlock))
            atomicOr(cluster.map_shared_rank(&row[word - owner * chunk], owner), 1u << (id & 31));
        }
      }
    }
    __threadfence();           // queued tokens are visible to the block that walks them
    cluster.sync();            // every remote OR has landed
    if (sh_slow) {             // (the same in every block of the cluster)
      if (rank == 0 && threadIdx.x == 0) {
        const bool ok = run_slow_walks(mw, g, v, hist, [&](int id) {
          const int word = id >> 5, owner = word / chunk;
          if (XG_BOUND(word, v.n_words, kBoundRowWord) && XG_BOUND(owner, n_blocks, kBoundClusterBlock))
            atomicOr(cluster.map_shared_rank(&row[word - owner * chunk], owner), 1u << (id & 31));
        });
        if (!ok) fail_everywhere();
      }
      cluster.sync();
    }
  } else __syncthreads();
  // 3. write the slice
  const int failed = (total > 0 || fallback) ? sh_fail : 0;
  const bool clear = st0 != 0 || failed;
  for (int w = threadIdx.x; w < nw; w += blockDim.x) bitmask[(long long)b * row_stride + w0 + w] = clear ? 0 : (int32_t)row[w];
  if (rank == 0 && threadIdx.x == 0 && status_user) status_user[b] = st0 != 0 ? st0 : (failed ? -6 : 0);
  // 4. mask this slice of the request's logits (nobody writes `row` any more: every remote OR landed before the barrier)
  if (kApplyElems != 0 && nw > 0) {
    constexpr int kE = kApplyElems == 0 ? 8 : kApplyElems;
    void* row_base = kE == 8 ? (void*)((uint16_t*)logits + (long long)b * logits_row_stride_elems) : (void*)((uint32_t*)logits + (long long)b * logits_row_stride_elems);
    auto word_at = [&](int w) { return clear ? 0u : row[w - w0]; };
    apply_vectors<kE>((uint4*)row_base, w0 * 32 / kE, min(v.vocab_size / kE, w1 * 32 / kE), threadIdx.x, blockDim.x, word_at);
    if (w1 == v.n_words) apply_ragged_tail<kE>(row_base, v.vocab_size, threadIdx.x, blockDim.x, word_at);
  }
}

}  // namespace xg
