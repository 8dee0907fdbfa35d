// Warp-cooperative Earley primitives (Section 3.2 of the paper: scan, complete, predict) on
// sparse item lists.  One warp owns one set under construction; its lanes stride over items.
//
// An item is one uint32: (origin << 16) | dotted-rule id.  Moving the dot is "+1" on the id.
// A set under construction lives in `cur` with a small open-addressing hash for uniqueness
// (Section 3.2: an Earley set holds every item once).  Rules that derive the empty string never
// appear as items: every item whose post-dot non-terminal is nullable is accompanied by the
// item with the dot moved over it (table `skip`), and prediction uses precomputed closures.
#pragma once
#include <cuda_runtime.h>

#include "device_tables.h"
#include "host_tables.h"

namespace fmt {

constexpr uint32_t FULL = 0xffffffffu;
constexpr uint32_t EMPTY_SLOT = 0xffffffffu;

__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31u; }

__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16;
  x *= 0x7feb352du;
  x ^= x >> 15;
  x *= 0x846ca68bu;
  x ^= x >> 16;
  return x;
}

// per-warp counters kept in shared memory
enum : uint32_t { W_NCUR = 0, W_OVERFLOW = 1, W_NPAIRS = 2, W_ACCEPT = 3, W_CTRS = 8 };

struct WarpCtx {
  uint32_t* cur;        // items of the set under construction (shared or global memory)
  uint32_t cur_cap;
  uint32_t* hset;       // uniqueness hash, all EMPTY_SLOT between uses
  uint32_t hset_mask;   // slots - 1 (power of two)
  uint32_t* nt;         // [2*Nw] shared: non-terminals after a dot, then their prediction closure
  uint32_t* ctr;        // [W_CTRS] shared
};

// 1 inserted, 0 already there, -1 table full
__device__ __forceinline__ int hset_insert(uint32_t* hset, uint32_t mask, uint32_t key) {
  uint32_t h = mix32(key) & mask;
  for (uint32_t probe = 0; probe <= mask; ++probe) {
    uint32_t old = atomicCAS(&hset[h], EMPTY_SLOT, key);
    if (old == EMPTY_SLOT) return 1;
    if (old == key) return 0;
    h = (h + 1) & mask;
  }
  return -1;
}

__device__ __forceinline__ void hset_clear_all(uint32_t* hset, uint32_t mask) {
  __syncwarp();
  for (uint32_t i = lane_id(); i <= mask; i += 32) hset[i] = EMPTY_SLOT;
  __syncwarp();
}

// Remove the first `n` items of cur from the hash (they are exactly its contents).
__device__ __forceinline__ void hset_clear_items(const WarpCtx& w, uint32_t n) {
  __syncwarp();
  if (n * 8u > w.hset_mask) {
    hset_clear_all(w.hset, w.hset_mask);
    return;
  }
  for (uint32_t i = lane_id(); i < n; i += 32) {
    uint32_t key = w.cur[i];
    uint32_t h = mix32(key) & w.hset_mask;
    for (uint32_t probe = 0; probe <= w.hset_mask; ++probe) {
      if (w.hset[h] == key) {
        w.hset[h] = EMPTY_SLOT;
        break;
      }
      h = (h + 1) & w.hset_mask;
    }
  }
  __syncwarp();
}

// Add item `key` and the items reached by moving the dot over nullable non-terminals.
// May be called by any subset of lanes.
__device__ __forceinline__ void add_item(const GrammarDev& G, const WarpCtx& w, uint32_t key) {
  uint32_t n = (G.info[key & 0xFFFFu] >> INFO_SKIP_SHIFT) & INFO_SKIP_MASK;
  for (uint32_t j = 0; j <= n; ++j) {
    int r = hset_insert(w.hset, w.hset_mask, key + j);
    if (r == 1) {
      uint32_t idx = atomicAdd(&w.ctr[W_NCUR], 1u);
      if (idx < w.cur_cap) w.cur[idx] = key + j;
      else w.ctr[W_OVERFLOW] = 1u;
    } else if (r < 0) {
      w.ctr[W_OVERFLOW] = 1u;
    }
  }
}

__device__ __forceinline__ bool class_has(const GrammarDev& G, uint32_t cls, uint32_t byte) {
  return (G.class_bits[cls * 8u + (byte >> 5)] >> (byte & 31u)) & 1u;
}

// What scanning `byte` makes of item `it` (Section 3.2's Scan; `inf` = its info word): up to two items.
// An item before a terminal that matches moves its dot.  An item inside an automaton (a regular
// non-terminal, Section 4.1) follows the automaton's transition: it becomes the next state's item if that
// state has transitions of its own, and the completed item of the non-terminal if that state accepts (a
// state that accepts and leads nowhere is thus never an item: a finished automaton is dropped at once).
struct Scanned {
  uint32_t a, b;   // the items (valid if has_a / has_b)
  bool has_a, has_b;
};
__device__ __forceinline__ Scanned scan_item(const GrammarDev& G, uint32_t it, uint32_t inf, uint32_t byte) {
  Scanned r{0u, 0u, false, false};
  const uint32_t kind = inf >> INFO_KIND_SHIFT;
  if (kind == KIND_TERM) {
    r.has_a = class_has(G, inf & INFO_ARG_MASK, byte);
    r.a = it + 1u;
  } else if (kind == KIND_DFA) {
    const uint32_t g = inf & INFO_ARG_MASK;
    const uint32_t t = __ldg(&G.dfa_trans[(size_t)g * G.n_eq + G.eq_of_byte[byte]]);
    if (t != 0xFFFFu) {
      r.has_a = (t & 0x4000u) != 0u;
      r.a = (it & 0xFFFF0000u) | (G.dfa_first + (t & 0x3FFFu));
      r.has_b = (t & 0x8000u) != 0u;
      r.b = (it & 0xFFFF0000u) | __ldg(&G.dfa_done[g]);
    }
  }
  return r;
}

// Scan (Section 3.2): items of `set` whose post-dot terminal matches `byte`, dot advanced, go
// into cur.  Returns the number of items in cur afterwards (uniform over the warp).
__device__ __forceinline__ uint32_t scan_into_cur(const GrammarDev& G, const WarpCtx& w, const uint32_t* set,
                                                  uint32_t len, uint32_t byte) {
  for (uint32_t k = lane_id(); k < len; k += 32) {
    uint32_t it = set[k];
    uint32_t inf = G.info[it & 0xFFFFu];
    const Scanned sc = scan_item(G, it, inf, byte);
    if (sc.has_a) add_item(G, w, sc.a);
    if (sc.has_b) add_item(G, w, sc.b);
  }
  __syncwarp();
  return min(w.ctr[W_NCUR], w.cur_cap);
}

// Complete (Section 3.2) to a fixpoint over cur, starting at item index `head`.  `view(o, ptr, len)`
// yields the items of set o and `view.fix(item, o)` rewrites an item read from set o into the
// naming used by the set under construction (identity for plain charts).  Completed items whose origin is the set itself are not processed:
// they can only come from empty derivations, already covered by `skip`.  Non-terminals found
// after a dot are collected in w.nt[0..Nw) for the prediction that follows; the accept item is
// reported in ctr[W_ACCEPT].
template <class View>
__device__ __forceinline__ void complete_fixpoint(const GrammarDev& G, const WarpCtx& w, const View& view,
                                                  uint32_t cur_index, uint32_t head) {
  const uint32_t lane = lane_id();
  for (;;) {
    __syncwarp();
    uint32_t n = min(w.ctr[W_NCUR], w.cur_cap);
    uint32_t over = w.ctr[W_OVERFLOW];
    __syncwarp();
    if (head >= n || over) break;
    uint32_t idx = head + lane;
    bool have = idx < n;
    uint32_t it = have ? w.cur[idx] : 0u;
    uint32_t inf = have ? G.info[it & 0xFFFFu] : 0u;
    uint32_t kind = inf >> INFO_KIND_SHIFT;
    if (have && kind == KIND_NT) {
      uint32_t y = inf & INFO_ARG_MASK;
      atomicOr(&w.nt[y >> 5], 1u << (y & 31u));
    }
    if (have && kind == KIND_END && (it & 0xFFFFu) == ITEM_ACCEPT) w.ctr[W_ACCEPT] = 1u;
    bool done_item = have && kind == KIND_END && (it >> 16) != cur_index && (it & 0xFFFFu) != ITEM_ACCEPT;  // (nothing waits for the augmented start symbol)
    uint32_t bal = __ballot_sync(FULL, done_item);
    while (bal) {
      int src = __ffs(bal) - 1;
      bal &= bal - 1;
      uint32_t X = __shfl_sync(FULL, inf & INFO_ARG_MASK, src);
      uint32_t o = __shfl_sync(FULL, it >> 16, src);
      const uint32_t* sp;
      uint32_t sl;
      view(o, sp, sl);
      for (uint32_t k = lane; k < sl; k += 32) {
        uint32_t wi = sp[k];
        uint32_t winf = G.info[wi & 0xFFFFu];
        if ((winf >> INFO_KIND_SHIFT) == KIND_NT && (winf & INFO_ARG_MASK) == X) add_item(G, w, view.fix(wi, o) + 1u);
      }
      __syncwarp();
    }
    head = min(head + 32u, n);  // items appended during this wave start at index n
  }
  __syncwarp();
}

// Predict (Section 3.2) for all non-terminals collected in w.nt[0..Nw): append the start items of
// every rule of every non-terminal in their closure, origin = cur_index.  These items are all new
// (nothing else in the set has this origin), so no uniqueness check is needed.  One closure word
// (32 non-terminals) per pass: a warp scan gives every lane the place of its non-terminal's items;
// short lists are copied by their lane, long ones (alternations of many literals) by the whole warp.
__device__ __forceinline__ void predict_into_cur(const GrammarDev& G, const WarpCtx& w, uint32_t cur_index) {
  const uint32_t lane = lane_id();
  const uint32_t Nw = G.Nw;
  uint32_t* ntmask = w.nt;
  uint32_t* clos = w.nt + Nw;
  __syncwarp();
  for (uint32_t i = lane; i < Nw; i += 32) {  // each lane owns some words of the closure
    uint32_t acc = 0u;
    for (uint32_t wi = 0; wi < Nw; ++wi) {
      uint32_t bits = ntmask[wi];
      while (bits) {
        const uint32_t y = wi * 32u + (uint32_t)(__ffs(bits) - 1);
        bits &= bits - 1;
        acc |= G.nt_closure[y * Nw + i];
      }
    }
    clos[i] = acc;
  }
  __syncwarp();
  uint32_t n = min(w.ctr[W_NCUR], w.cur_cap);
  bool over = false;
  for (uint32_t wi = 0; wi < Nw; ++wi) {
    const uint32_t bits = clos[wi];
    if (bits == 0u) continue;  // (uniform) most words of the closure are empty
    uint32_t lo = 0, len = 0;
    if ((bits >> lane) & 1u) {
      const uint32_t z = wi * 32u + lane;
      lo = G.direct_off[z];
      len = G.direct_off[z + 1] - lo;
    }
    uint32_t incl = len;
    for (int d = 1; d < 32; d <<= 1) {
      uint32_t t = __shfl_up_sync(FULL, incl, d);
      if ((int)lane >= d) incl += t;
    }
    const uint32_t total = __shfl_sync(FULL, incl, 31);
    if (n + total > w.cur_cap) {
      over = true;
      break;
    }
    const uint32_t at = n + incl - len;
    const bool is_long = len > 8u;
    if (!is_long)
      for (uint32_t i = 0; i < len; ++i) w.cur[at + i] = (cur_index << 16) | (uint32_t)G.direct_items[lo + i];
    uint32_t longs = __ballot_sync(FULL, is_long);
    while (longs) {
      const int src = __ffs(longs) - 1;
      longs &= longs - 1;
      const uint32_t slo = __shfl_sync(FULL, lo, src), slen = __shfl_sync(FULL, len, src), sat = __shfl_sync(FULL, at, src);
      for (uint32_t i = lane; i < slen; i += 32) w.cur[sat + i] = (cur_index << 16) | (uint32_t)G.direct_items[slo + i];
    }
    n += total;
  }
  __syncwarp();
  if (lane == 0) {
    w.ctr[W_NCUR] = n;
    if (over) w.ctr[W_OVERFLOW] = 1u;
  }
  for (uint32_t i = lane; i < Nw; i += 32) ntmask[i] = 0u;
  __syncwarp();
}

// Is `key` in the uniqueness hash?
__device__ __forceinline__ bool hset_contains(const uint32_t* hset, uint32_t mask, uint32_t key) {
  uint32_t h = mix32(key) & mask;
  for (uint32_t probe = 0; probe <= mask; ++probe) {
    const uint32_t v = hset[h];
    if (v == key) return true;
    if (v == EMPTY_SLOT) return false;
    h = (h + 1) & mask;
  }
  return false;
}

__device__ __forceinline__ void clear_nt(const GrammarDev& G, const WarpCtx& w) {
  __syncwarp();
  for (uint32_t i = lane_id(); i < 2 * G.Nw; i += 32) w.nt[i] = 0u;
  __syncwarp();
}

// ---- The lane-resident form of Scan and Complete, for sets of at most 32 items: the set under
// construction sits one item per lane, uniqueness is a matter of shuffles and
// ballots, and neither the uniqueness hash nor a shared-memory counter is touched.
constexpr uint32_t SMALL_OVERFLOW = 0xffffffffu;

// The candidates c .. c + skip of the lanes with `v` set join the set unless already there.  The
// set sits one item per lane: `mine` is item `lane` for lane < n.  One candidate at a time (there
// are seldom more than one or two per call): a broadcast, and a ballot of "is it mine?".  Returns
// the new count, above 32 when they do not fit.
__device__ __forceinline__ uint32_t append_small(uint32_t c, bool v, uint32_t skip, uint32_t n, uint32_t& mine) {
  const uint32_t lane = lane_id();
  uint32_t vm = __ballot_sync(FULL, v);
  while (vm) {
    const int src = __ffs(vm) - 1;
    vm &= vm - 1;
    const uint32_t c0 = __shfl_sync(FULL, c, src), sk = __shfl_sync(FULL, skip, src);
    for (uint32_t j = 0; j <= sk; ++j) {
      const uint32_t cj = c0 + j;
      if (__ballot_sync(FULL, lane < n && mine == cj)) continue;  // already there
      if (n == 32u) return 33u;
      if (lane == n) mine = cj;
      ++n;
    }
  }
  return n;
}

// Scan the items of `set` over `byte`, then Complete to a fixpoint (Section 3.2), all in lanes.
// `rename(item)` rewrites an item of `set` into the naming of the new set (identity for plain
// charts); `view` and `cur_index` are as for complete_fixpoint.  On return the lanes' `mine`
// hold the n <= 32 items (completed ones included), the non-terminals found after a
// dot are collected in w.nt[0..Nw), and `accept` tells whether the accept item is among them.
// Returns n (0: the byte cannot follow), or SMALL_OVERFLOW when the set outgrows 32 items (w.nt is
// clean then and the caller takes the general path).
template <class View, class Rename>
__device__ __forceinline__ uint32_t small_scan_complete(const GrammarDev& G, const WarpCtx& w, const View& view,
                                                        const uint32_t* set, uint32_t len, uint32_t byte, uint32_t cur_index,
                                                        Rename rename, uint32_t& mine, bool& accept) {
  const uint32_t lane = lane_id();
  uint32_t n = 0;
  mine = 0;
  accept = false;
  __syncwarp();
  for (uint32_t base = 0; base < len; base += 32) {
    const uint32_t k = base + lane;
    uint32_t it = k < len ? set[k] : 0u;
    const uint32_t inf = k < len ? G.info[it & 0xFFFFu] : 0u;  // (info word 0 is a non-terminal item: scans nothing)
    it = rename(it);
    const Scanned sc = scan_item(G, it, k < len ? inf : (KIND_NT << INFO_KIND_SHIFT), byte);
    const uint32_t skip_a = sc.has_a ? (G.info[sc.a & 0xFFFFu] >> INFO_SKIP_SHIFT) & INFO_SKIP_MASK : 0u;
    if (__any_sync(FULL, sc.has_a)) n = append_small(sc.a, sc.has_a, skip_a, n, mine);
    if (n > 32u) return SMALL_OVERFLOW;
    if (__any_sync(FULL, sc.has_b)) n = append_small(sc.b, sc.has_b, 0u, n, mine);  // (a completed item has nothing to skip)
    if (n > 32u) return SMALL_OVERFLOW;
  }
  if (n == 0) return 0;
  uint32_t head = 0;  // lanes [head, n) hold the items not looked at yet
  while (head < n) {
    const bool have = lane >= head && lane < n;
    const uint32_t inf = have ? G.info[mine & 0xFFFFu] : 0u;
    const uint32_t kind = inf >> INFO_KIND_SHIFT;
    if (have && kind == KIND_NT) {
      const uint32_t y = inf & INFO_ARG_MASK;
      atomicOr(&w.nt[y >> 5], 1u << (y & 31u));
    }
    if (__any_sync(FULL, have && kind == KIND_END && (mine & 0xFFFFu) == ITEM_ACCEPT)) accept = true;
    uint32_t bal = __ballot_sync(FULL, have && kind == KIND_END && (mine >> 16) != cur_index && (mine & 0xFFFFu) != ITEM_ACCEPT);
    const uint32_t it = mine;
    head = n;
    while (bal) {
      const int src = __ffs(bal) - 1;
      bal &= bal - 1;
      const uint32_t X = __shfl_sync(FULL, inf & INFO_ARG_MASK, src);
      const uint32_t o = __shfl_sync(FULL, it >> 16, src);
      const uint32_t* sp;
      uint32_t sl;
      view(o, sp, sl);
      for (uint32_t base = 0; base < sl; base += 32) {
        const uint32_t k = base + lane;
        const uint32_t wi = k < sl ? sp[k] : 0u;
        const uint32_t winf = k < sl ? G.info[wi & 0xFFFFu] : 0u;
        const bool match = (winf >> INFO_KIND_SHIFT) == KIND_NT && (winf & INFO_ARG_MASK) == X;
        const uint32_t cand = view.fix(wi, o) + 1u;
        const uint32_t skip = match ? (G.info[cand & 0xFFFFu] >> INFO_SKIP_SHIFT) & INFO_SKIP_MASK : 0u;
        if (__any_sync(FULL, match)) n = append_small(cand, match, skip, n, mine);
        if (n > 32u) {
          clear_nt(G, w);
          return SMALL_OVERFLOW;
        }
      }
    }
  }
  return n;
}

// Drop the completed items of a lane-resident set: the others move to cur[0..count) and to the
// first lanes' `mine`.  Returns their count.
__device__ __forceinline__ uint32_t small_drop_completed(const GrammarDev& G, const WarpCtx& w, uint32_t n, uint32_t& mine) {
  const uint32_t lane = lane_id();
  const bool keep = lane < n && (G.info[mine & 0xFFFFu] >> INFO_KIND_SHIFT) != KIND_END;
  const uint32_t kb = __ballot_sync(FULL, keep);
  __syncwarp();
  if (keep) w.cur[__popc(kb & ((1u << lane) - 1u))] = mine;
  __syncwarp();
  const uint32_t nk = __popc(kb);
  mine = lane < nk ? w.cur[lane] : 0u;
  return nk;
}

// Copy the grammar's hot tables into shared memory (all threads of the block take part, the
// caller synchronizes) and return a view of the grammar that reads them from there.
__device__ __forceinline__ GrammarDev stage_hot_tables(const GrammarDev& Gg, uint32_t* dst) {
  for (uint32_t i = threadIdx.x; i < Gg.hot_words; i += blockDim.x) dst[i] = Gg.hot_block[i];
  GrammarDev G = Gg;
  G.info = dst + (Gg.info - Gg.hot_block);
  G.class_bits = dst + (Gg.class_bits - Gg.hot_block);
  G.eq_of_byte = reinterpret_cast<const uint8_t*>(dst + (reinterpret_cast<const uint32_t*>(Gg.eq_of_byte) - Gg.hot_block));
  G.nt_closure = dst + (Gg.nt_closure - Gg.hot_block);
  G.direct_off = dst + (Gg.direct_off - Gg.hot_block);
  G.direct_items = reinterpret_cast<const uint16_t*>(dst + (reinterpret_cast<const uint32_t*>(Gg.direct_items) - Gg.hot_block));
  G.hot_block = dst;
  return G;
}

// Drop the items with the dot at the end from cur[0..n) in place; returns the new count.
__device__ __forceinline__ uint32_t drop_completed(const GrammarDev& G, const WarpCtx& w, uint32_t n) {
  const uint32_t lane = lane_id();
  uint32_t out = 0;
  __syncwarp();
  for (uint32_t base = 0; base < n; base += 32) {
    uint32_t idx = base + lane;
    bool have = idx < n;
    uint32_t it = have ? w.cur[idx] : 0u;
    bool keep = have && (G.info[it & 0xFFFFu] >> INFO_KIND_SHIFT) != KIND_END;
    uint32_t bal = __ballot_sync(FULL, keep);
    uint32_t pos = out + __popc(bal & ((1u << lane) - 1u));
    __syncwarp();
    if (keep) w.cur[pos] = it;
    out += __popc(bal);
    __syncwarp();
  }
  return out;
}

// OR of the byte classes of all post-dot terminals of a set: the bytes that can be scanned.
__device__ __forceinline__ void scannable_bytes(const GrammarDev& G, const uint32_t* set, uint32_t len,
                                                uint32_t* out8 /* shared */) {
  uint32_t acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0u;
  for (uint32_t k = lane_id(); k < len; k += 32) {
    uint32_t inf = G.info[set[k] & 0xFFFFu];
    const uint32_t kind = inf >> INFO_KIND_SHIFT;
    if (kind == KIND_TERM || kind == KIND_DFA) {
      const uint4* p = reinterpret_cast<const uint4*>(kind == KIND_TERM ? G.class_bits + (inf & INFO_ARG_MASK) * 8u
                                                                        : G.dfa_scan + (size_t)(inf & INFO_ARG_MASK) * 8u);
      uint4 a = p[0], b = p[1];
      acc[0] |= a.x, acc[1] |= a.y, acc[2] |= a.z, acc[3] |= a.w;
      acc[4] |= b.x, acc[5] |= b.y, acc[6] |= b.z, acc[7] |= b.w;
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = __reduce_or_sync(FULL, acc[i]);
  __syncwarp();
  if (lane_id() == 0) {
#pragma unroll
    for (int i = 0; i < 8; ++i) out8[i] = acc[i];
  }
  __syncwarp();
}

// Ascending bitonic sort of a[0..n); the array must have room for the next power of two >= max(n, 32),
// which must not exceed cap_pow2.
__device__ __forceinline__ void sort_items(uint32_t* a, uint32_t n, uint32_t cap_pow2) {
  const uint32_t lane = lane_id();
  if (n <= 32) {  // one item per lane, compare-exchange through shuffles
    __syncwarp();
    uint32_t v = (lane < n) ? a[lane] : 0xffffffffu;
#pragma unroll
    for (uint32_t k = 2; k <= 32; k <<= 1) {
#pragma unroll
      for (uint32_t j = k >> 1; j > 0; j >>= 1) {
        const uint32_t other = __shfl_xor_sync(FULL, v, j);
        const bool up = (lane & k) == 0, lower = (lane & j) == 0;
        v = (lower == up) ? min(v, other) : max(v, other);
      }
    }
    if (lane < n) a[lane] = v;
    __syncwarp();
    return;
  }
  uint32_t P = 32;
  while (P < n) P <<= 1;
  if (P > cap_pow2) P = cap_pow2;
  __syncwarp();
  for (uint32_t i = n + lane; i < P; i += 32) a[i] = 0xffffffffu;
  __syncwarp();
  for (uint32_t k = 2; k <= P; k <<= 1) {
    for (uint32_t j = k >> 1; j > 0; j >>= 1) {
      for (uint32_t i = lane; i < P; i += 32) {
        uint32_t l = i ^ j;
        if (l > i) {
          uint32_t x = a[i], y = a[l];
          bool up = (i & k) == 0;
          if ((x > y) == up) {
            a[i] = y;
            a[l] = x;
          }
        }
      }
      __syncwarp();
    }
  }
}

}  // namespace fmt
