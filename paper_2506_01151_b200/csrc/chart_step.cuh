// One token on a whole pruned chart, by one warp (used when a sequence advances).  Per byte:
//   Scan -> Complete (fixpoint) -> Predict; after the token's last byte: Compact (Section 4.2.3),
// which leaves exactly the chart that compacting after every byte would leave (an item needed at
// the end was needed at every step before), at a fraction of the work,
// and the state cache: the pruned chart, densely renumbered, is the cache key (Section 5.2: token
// sequences that differ may still end in one and the same pruned chart, and then share an entry).
//
// Compact keeps, besides the unfinished items of the new last set, exactly the items a later
// Complete can still read: an item (Y -> mu . A nu, o') of an earlier set o stays iff a kept item
// with left-hand side A and origin o exists (Figure 3: sets not on a reference chain of the last
// set's items are removed; completed items go once their set is done).
#pragma once
#include "earley_device.cuh"

namespace fmt {

constexpr uint32_t ADV_CUR_CAP = 2048;     // items of the sets a token adds to a chart (shared-memory arena)
constexpr uint32_t ADV_HSET = 2048;        // hash slots (power of two)
constexpr uint32_t ADV_MAX_ITEMS = 65536;  // items of a chart the live bitmap can describe
constexpr uint32_t ADV_PAIRS = 1024;       // (set, non-terminal) needs of one Compact
constexpr uint32_t ADV_MAX_SETS = 2048;
constexpr uint32_t ADV_NT_WORDS = 256;     // 2 * Nw, Nw <= 128
constexpr uint32_t ADV_STAGE = 2048;       // a source chart up to this many words is read from shared memory
constexpr uint32_t ADV_WARP_WORDS =
    ADV_CUR_CAP + ADV_HSET + ADV_MAX_ITEMS / 32 + ADV_PAIRS + ADV_MAX_SETS + ADV_NT_WORDS + W_CTRS + ADV_STAGE;

struct AdvScratch {
  WarpCtx w;
  uint32_t* live;   // [ADV_MAX_ITEMS/32] bitmap over the source chart's items
  uint32_t* pairs;  // [ADV_PAIRS]
  uint32_t* sets;   // [ADV_MAX_SETS] per-set live count, then new index
  uint32_t* stage;  // [ADV_STAGE]
};

__device__ __forceinline__ AdvScratch adv_scratch(uint32_t* base) {
  AdvScratch s;
  s.w.cur = base;
  s.w.cur_cap = ADV_CUR_CAP;
  s.w.hset = base + ADV_CUR_CAP;
  s.w.hset_mask = ADV_HSET - 1;
  s.live = s.w.hset + ADV_HSET;
  s.pairs = s.live + ADV_MAX_ITEMS / 32;
  s.sets = s.pairs + ADV_PAIRS;
  s.w.nt = s.sets + ADV_MAX_SETS;
  s.w.ctr = s.w.nt + ADV_NT_WORDS;
  s.stage = s.w.ctr + W_CTRS;
  return s;
}

struct ChartView {
  const uint32_t* off;  // set_off
  const uint32_t* items;
  __device__ __forceinline__ void operator()(uint32_t o, const uint32_t*& p, uint32_t& n) const {
    uint32_t a = off[o], b = off[o + 1];
    p = items + a;
    n = b - a;
  }
  __device__ __forceinline__ uint32_t fix(uint32_t item, uint32_t) const { return item; }
};

__device__ __forceinline__ void push_need(const AdvScratch& s, uint32_t o, uint32_t A) {
  uint32_t key = (o << 16) | A;
  int r = hset_insert(s.w.hset, s.w.hset_mask, key);
  if (r == 0) return;  // already asked for
  // r < 0 (hash full): ask again anyway, a repeated need only costs time
  uint32_t idx = atomicAdd(&s.w.ctr[W_NPAIRS], 1u);
  if (idx < ADV_PAIRS) s.pairs[idx] = key;
  else s.w.ctr[W_OVERFLOW] = 1u;
}

// The chart hash is a sum over (word index, value) pairs, so it can be accumulated while the
// words are written, in any order and by any lane.  Two independent 32-bit sums.
struct HashAcc {
  uint32_t h1 = 0, h2 = 0;
  __device__ __forceinline__ void add(uint32_t i, uint32_t v) {
    h1 += mix32(v ^ (i * 0x9E3779B1u));
    h2 += mix32((v + 0x632BE5ABu) ^ (i * 0x85EBCA77u));
  }
};
__device__ __forceinline__ void put(uint32_t* ch, HashAcc& h, uint32_t i, uint32_t v) {
  ch[i] = v;
  h.add(i, v);
}

// Write the last set (cur[0..n), unsorted, completed items already removed) and finish the header.
// dst already holds set_off[0..m_new) and the kept items of the earlier sets (`kept` of them), all
// accounted for in `h`.
__device__ __forceinline__ int finish_chart(const AdvScratch& s, uint32_t* dst, uint32_t dst_cap, uint32_t m_new,
                                            uint32_t kept, uint32_t n, bool accepting, HashAcc h) {
  const uint32_t lane = lane_id();
  uint32_t words = CH_HDR + (m_new + 2) + kept + n;
  if (words > dst_cap || kept + n >= ADV_MAX_ITEMS) return -1;
  sort_items(s.w.cur, n, 1u << 30);
  const uint32_t items_at = CH_HDR + (m_new + 2);
  for (uint32_t i = lane; i < n; i += 32) put(dst, h, items_at + kept + i, s.w.cur[i]);
  if (lane == 0) {
    put(dst, h, CH_SETS, m_new + 1);
    put(dst, h, CH_ITEMS, kept + n);
    put(dst, h, CH_FLAGS, accepting ? CHART_ACCEPTING : 0u);
    put(dst, h, CH_WORDS, words);
    put(dst, h, 6, 0u);
    put(dst, h, 7, 0u);
    put(dst, h, CH_HDR + m_new, kept);          // first item of the last set
    put(dst, h, CH_HDR + m_new + 1, kept + n);  // end
  }
  for (int d = 16; d > 0; d >>= 1) {
    h.h1 += __shfl_xor_sync(FULL, h.h1, d);
    h.h2 += __shfl_xor_sync(FULL, h.h2, d);
  }
  if (lane == 0) {
    dst[CH_HASH_LO] = h.h1;
    dst[CH_HASH_HI] = h.h2;
  }
  __syncwarp();
  return 1;
}

// The start chart: S[0] = closure of ($ -> . start, 0).
__device__ int chart_init(const GrammarDev& G, const AdvScratch& s, uint32_t* dst, uint32_t dst_cap) {
  const uint32_t lane = lane_id();
  if (lane < W_CTRS) s.w.ctr[lane] = 0u;
  clear_nt(G, s.w);
  if (lane == 0) add_item(G, s.w, ITEM_START);
  __syncwarp();
  ChartView none{nullptr, nullptr};
  complete_fixpoint(G, s.w, none, 0u, 0u);  // only collects post-dot non-terminals and the accept flag
  uint32_t hashed = min(s.w.ctr[W_NCUR], s.w.cur_cap);
  bool accepting = s.w.ctr[W_ACCEPT] != 0u;
  hset_clear_items(s.w, hashed);
  predict_into_cur(G, s.w, 0u);
  if (s.w.ctr[W_OVERFLOW]) {
    hset_clear_all(s.w.hset, s.w.hset_mask);
    clear_nt(G, s.w);
    return -1;
  }
  uint32_t n = drop_completed(G, s.w, min(s.w.ctr[W_NCUR], s.w.cur_cap));
  return finish_chart(s, dst, dst_cap, 0u, 0u, n, accepting, HashAcc{});
}

// Where set o of "source chart + the token's sets so far" lives.  Sets 0..m-1 are the source
// chart's, set m-1+L is the token's L-th.
struct TokenView {
  const uint32_t* soff;
  const uint32_t* sitems;
  uint32_t m;
  const uint32_t* arena;
  const uint32_t* lvl_off;  // [MAX_TOKEN_BYTES + 2] first item of each level in the arena
  __device__ __forceinline__ void operator()(uint32_t o, const uint32_t*& p, uint32_t& n) const {
    if (o < m) {
      uint32_t a = soff[o], b = soff[o + 1];
      p = sitems + a;
      n = b - a;
    } else {
      const uint32_t L = o - (m - 1);
      p = arena + lvl_off[L];
      n = lvl_off[L + 1] - lvl_off[L];
    }
  }
  __device__ __forceinline__ uint32_t fix(uint32_t item, uint32_t) const { return item; }
  // position of item k of set o in the live bitmap (source items first, then the arena)
  __device__ __forceinline__ uint32_t bit_base(uint32_t o, uint32_t n_items) const {
    return (o < m) ? soff[o] : n_items + lvl_off[o - (m - 1)];
  }
};

// All bytes of one token.  Returns 1 (dst holds the new chart), 0 (some byte cannot follow: dst
// is garbage), -1 (a capacity limit was hit) or -2 (the arena for the token's sets is too small:
// the caller may retry with a larger one).  src and dst must not overlap.  `arena` (arena_cap
// items, a power of two if the last set is to be sorted in place) holds the token's sets.
//
// With `forced_out` set, the bytes are not given but found: as long as the text so far is not a sentence and
// exactly one byte can follow, that byte is taken (and written to forced_out); `len` is then the longest run
// looked for, nothing is compacted or written to dst, and the return value is the length of the run.
__device__ int token_step(const GrammarDev& G, AdvScratch& s, const uint32_t* src, const uint8_t* bytes, uint32_t len,
                          uint32_t* dst, uint32_t dst_cap, uint32_t* arena, uint32_t arena_cap,
                          uint8_t* forced_out = nullptr) {
  const uint32_t lane = lane_id();
  const uint32_t m = src[CH_SETS];
  const uint32_t n_items = src[CH_ITEMS];
  if (m == 0 || m + len + MAX_TOKEN_BYTES + 4 > ADV_MAX_SETS || n_items > ADV_MAX_ITEMS || len > MAX_TOKEN_BYTES)
    return forced_out ? 0 : -1;
  // small charts are read from shared memory from here on
  const uint32_t src_words = src[CH_WORDS];
  __syncwarp();
  if (src_words <= ADV_STAGE) {
    for (uint32_t i = lane; i < src_words; i += 32) s.stage[i] = src[i];
    src = s.stage;
  }
  uint32_t* lvl_off = s.sets + ADV_MAX_SETS - (MAX_TOKEN_BYTES + 2);  // the tail of `sets` is free until Compact ends
  TokenView view{src + CH_HDR, src + CH_HDR + m + 1, m, arena, lvl_off};
  const uint32_t* soff = view.soff;
  const uint32_t* sitems = view.sitems;
  if (lane == 0) lvl_off[0] = 0, lvl_off[1] = 0;
  __syncwarp();
  // ---- per byte: Scan, Complete, Predict; the new set is appended to the arena
  uint32_t top = 0;
  bool accepting = forced_out != nullptr && (src[CH_FLAGS] & CHART_ACCEPTING) != 0u;
  const uint32_t* prev = sitems + soff[m - 1];
  uint32_t prev_len = soff[m] - soff[m - 1];
  for (uint32_t L = 1; L <= len; ++L) {
    if (top + 64 > arena_cap) return forced_out ? (int)(L - 1) : -2;
    uint32_t byte;
    if (forced_out) {  // is the next byte forced?
      if (accepting) return (int)(L - 1);  // the text may end here
      scannable_bytes(G, prev, prev_len, s.pairs);
      uint32_t wd = lane < 8 ? s.pairs[lane] : 0u;
      uint32_t cnt = __popc(wd);
      for (int dd = 16; dd > 0; dd >>= 1) cnt += __shfl_xor_sync(FULL, cnt, dd);
      if (cnt != 1u) return (int)(L - 1);
      const uint32_t has = __ballot_sync(FULL, wd != 0u);
      const int src_lane = __ffs(has) - 1;
      byte = (uint32_t)src_lane * 32u + (uint32_t)(__ffs(__shfl_sync(FULL, wd, src_lane)) - 1);
      __syncwarp();
    } else {
      byte = __ldg(&bytes[L - 1]);
    }
    s.w.cur = arena + top;
    s.w.cur_cap = arena_cap - top;
    __syncwarp();
    if (lane < W_CTRS) s.w.ctr[lane] = 0u;
    __syncwarp();
    const uint32_t index = m - 1 + L;
    uint32_t n;
    // sets of up to 32 scanned and completed items (nearly all) are built in lanes ...
    uint32_t mine;
    const uint32_t ns = (prev_len <= 96u) ? small_scan_complete(G, s.w, view, prev, prev_len, byte, index,
                                                                 [](uint32_t it) { return it; }, mine, accepting)
                                           : SMALL_OVERFLOW;
    if (ns == 0) return forced_out ? (int)(L - 1) : 0;
    if (ns != SMALL_OVERFLOW) {
      const uint32_t nk = small_drop_completed(G, s.w, ns, mine);
      if (lane == 0) s.w.ctr[W_NCUR] = nk;
      predict_into_cur(G, s.w, index);
      if (s.w.ctr[W_OVERFLOW]) return forced_out ? (int)(L - 1) : -2;
      n = min(s.w.ctr[W_NCUR], s.w.cur_cap);
    } else {  // ... larger ones with the uniqueness hash
      n = scan_into_cur(G, s.w, prev, prev_len, byte);
      if (s.w.ctr[W_OVERFLOW]) {
        hset_clear_all(s.w.hset, s.w.hset_mask);
        return forced_out ? (int)(L - 1) : -2;
      }
      if (n == 0) return forced_out ? (int)(L - 1) : 0;
      complete_fixpoint(G, s.w, view, index, 0u);
      uint32_t hashed = min(s.w.ctr[W_NCUR], s.w.cur_cap);
      if (s.w.ctr[W_OVERFLOW]) {
        hset_clear_all(s.w.hset, s.w.hset_mask);
        clear_nt(G, s.w);
        return forced_out ? (int)(L - 1) : -2;
      }
      hset_clear_items(s.w, hashed);
      accepting = s.w.ctr[W_ACCEPT] != 0u;
      predict_into_cur(G, s.w, index);
      if (s.w.ctr[W_OVERFLOW]) return forced_out ? (int)(L - 1) : -2;
      n = drop_completed(G, s.w, min(s.w.ctr[W_NCUR], s.w.cur_cap));
    }
    prev = arena + top;
    prev_len = n;
    top += n;
    if (lane == 0) lvl_off[L + 1] = top;
    if (forced_out && lane == 0) forced_out[L - 1] = (uint8_t)byte;  // (the step went through: the byte counts)
    __syncwarp();
  }
  if (forced_out) return (int)len;
  // ---- Compact once: which items of the earlier sets can a later Complete still read?
  const uint32_t last = m - 1 + len;           // index of the last set
  const uint32_t last_at = lvl_off[len];       // its first item in the arena
  const uint32_t n_last = top - last_at;
  const uint32_t n_bits = n_items + last_at;   // source items, then the token's earlier sets
  if (n_bits > ADV_MAX_ITEMS) return -1;
  for (uint32_t i = lane; i < (n_bits + 31) / 32; i += 32) s.live[i] = 0u;
  __syncwarp();
  for (uint32_t i = lane; i < n_last; i += 32) {
    uint32_t it = arena[last_at + i];
    if ((it >> 16) < last) push_need(s, it >> 16, __ldg(&G.lhs[it & 0xFFFFu]));
  }
  // needs are served a wave at a time: a need whose set is short is served by its own lane, the
  // needs of long sets (alternations of many literals predicted at once) by the whole warp in turn
  constexpr uint32_t NEED_SHORT = 8;
  for (uint32_t head = 0;;) {
    __syncwarp();
    const uint32_t np = min(s.w.ctr[W_NPAIRS], ADV_PAIRS);
    __syncwarp();
    if (head >= np) break;
    const uint32_t mine = head + lane;
    uint32_t o = 0, A = 0, sl = 0, base = 0;
    const uint32_t* sp = nullptr;
    if (mine < np) {
      const uint32_t key = s.pairs[mine];
      o = key >> 16, A = key & 0xFFFFu;
      view(o, sp, sl);
      base = view.bit_base(o, n_items);
    }
    auto serve = [&](const uint32_t* set, uint32_t k, uint32_t bit_base, uint32_t want) {
      const uint32_t wi = set[k];
      const uint32_t inf = G.info[wi & 0xFFFFu];
      if ((inf >> INFO_KIND_SHIFT) == KIND_NT && (inf & INFO_ARG_MASK) == want) {
        const uint32_t pos = bit_base + k;
        const uint32_t bit = 1u << (pos & 31u);
        const uint32_t old = atomicOr(&s.live[pos >> 5], bit);
        if (!(old & bit)) push_need(s, wi >> 16, __ldg(&G.lhs[wi & 0xFFFFu]));
      }
    };
    if (sl <= NEED_SHORT)
      for (uint32_t k = 0; k < sl; ++k) serve(sp, k, base, A);
    uint32_t longs = __ballot_sync(FULL, sl > NEED_SHORT);
    while (longs) {
      const int src = __ffs(longs) - 1;
      longs &= longs - 1;
      const uint32_t so = __shfl_sync(FULL, o, src), sA = __shfl_sync(FULL, A, src);
      const uint32_t* lp;
      uint32_t ll;
      view(so, lp, ll);
      const uint32_t lbase = view.bit_base(so, n_items);
      for (uint32_t k = lane; k < ll; k += 32) serve(lp, k, lbase, sA);
    }
    head = min(head + 32u, np);
  }
  const uint32_t n_pairs = min(s.w.ctr[W_NPAIRS], ADV_PAIRS);
  __syncwarp();
  if (n_pairs * 8u > s.w.hset_mask) {
    hset_clear_all(s.w.hset, s.w.hset_mask);  // the hash held (set, non-terminal) pairs
  } else {
    for (uint32_t i = lane; i < n_pairs; i += 32) {
      const uint32_t key = s.pairs[i];
      uint32_t hh = mix32(key) & s.w.hset_mask;
      for (uint32_t probe = 0; probe <= s.w.hset_mask; ++probe) {
        if (s.w.hset[hh] == key) {
          s.w.hset[hh] = EMPTY_SLOT;
          break;
        }
        hh = (hh + 1) & s.w.hset_mask;
      }
    }
    __syncwarp();
  }
  if (s.w.ctr[W_OVERFLOW]) {
    hset_clear_all(s.w.hset, s.w.hset_mask);
    clear_nt(G, s.w);
    return -1;
  }
  // ---- live items per earlier set, new set numbers, new offsets
  const uint32_t M = last;  // earlier sets: 0..last-1
  for (uint32_t k = lane; k < M; k += 32) {
    const uint32_t* sp;
    uint32_t sl;
    view(k, sp, sl);
    const uint32_t base = view.bit_base(k, n_items);
    uint32_t c = 0;
    for (uint32_t i = 0; i < sl; ++i) c += (s.live[(base + i) >> 5] >> ((base + i) & 31u)) & 1u;
    s.sets[k] = c;
  }
  __syncwarp();
  HashAcc h;
  uint32_t m_new = 0, kept = 0;
  for (uint32_t base = 0; base < M; base += 32) {
    uint32_t k = base + lane;
    uint32_t c = (k < M) ? s.sets[k] : 0u;
    uint32_t keep = __ballot_sync(FULL, c > 0);
    uint32_t my_new = m_new + __popc(keep & ((1u << lane) - 1u));
    uint32_t incl = c;  // inclusive prefix sum of the counts within the wave
    for (int d = 1; d < 32; d <<= 1) {
      uint32_t t = __shfl_up_sync(FULL, incl, d);
      if ((int)lane >= d) incl += t;
    }
    __syncwarp();
    if (k < M) {
      if (c > 0) {
        if (CH_HDR + my_new < dst_cap) put(dst, h, CH_HDR + my_new, kept + incl - c);
        s.sets[k] = my_new;
      } else {
        s.sets[k] = 0xffffffffu;
      }
    }
    kept += __shfl_sync(FULL, incl, 31);
    m_new += __popc(keep);
  }
  __syncwarp();
  if (CH_HDR + (m_new + 2) + kept + n_last + 64 > dst_cap) return -1;
  // ---- copy the live items (source chart first, then the token's earlier sets), origins renumbered
  const uint32_t items_at = CH_HDR + (m_new + 2);
  uint32_t bad = 0;
  uint32_t out = 0;
  for (uint32_t base = 0; base < n_bits; base += 32) {
    uint32_t i = base + lane;
    bool lv = (i < n_bits) && ((s.live[i >> 5] >> (i & 31u)) & 1u);
    uint32_t bal = __ballot_sync(FULL, lv);
    if (lv) {
      uint32_t it = (i < n_items) ? sitems[i] : arena[i - n_items];
      uint32_t no = s.sets[it >> 16];
      if (no == 0xffffffffu) bad = 1;
      const uint32_t at = items_at + out + __popc(bal & ((1u << lane) - 1u)), v = (no << 16) | (it & 0xFFFFu);
      if (i < n_items) put(dst, h, at, v);  // the source chart's sets are sorted and stay so
      else dst[at] = v;                     // the token's own sets are in the order they were built: sorted below
    }
    out += __popc(bal);
  }
  // ---- the kept items of the token's earlier sets, ascending like every other set: the chart is
  // the cache key, and the same bytes fed as other tokens must give the same words
  __syncwarp();
  for (uint32_t L = 1; L < len; ++L) {
    const uint32_t nw = s.sets[m - 1 + L];
    if (nw == 0xffffffffu) continue;  // (uniform)
    const uint32_t a = dst[CH_HDR + nw], b = (nw + 1 < m_new) ? dst[CH_HDR + nw + 1] : kept;
    uint32_t* set = dst + items_at + a;
    const uint32_t ns = b - a;
    if (ns <= 32) {
      sort_items(set, ns, 32);
    } else {  // rare: by rank, through the part of the arena whose sets have been copied out by now
      for (uint32_t i = lane; i < ns; i += 32) arena[i] = set[i];
      __syncwarp();
      for (uint32_t i = lane; i < ns; i += 32) {
        const uint32_t x = arena[i];
        uint32_t rank = 0;
        for (uint32_t k = 0; k < ns; ++k) rank += arena[k] < x ? 1u : 0u;
        set[rank] = x;  // (the items of a set are distinct)
      }
      __syncwarp();
    }
    for (uint32_t i = lane; i < ns; i += 32) h.add(items_at + a + i, set[i]);
  }
  // ---- the last set: renumber origins (its own index becomes m_new), move it to the front of the
  // arena region it occupies so that it can be sorted in place
  for (uint32_t i = lane; i < n_last; i += 32) {
    uint32_t it = arena[last_at + i];
    uint32_t o = it >> 16;
    uint32_t no = (o == last) ? m_new : s.sets[o];
    if (no == 0xffffffffu) bad = 1;
    arena[last_at + i] = (no << 16) | (it & 0xFFFFu);
  }
  bad = __any_sync(FULL, bad);
  __syncwarp();
  if (bad) return -1;
  uint32_t P = 32;
  while (P < n_last) P <<= 1;
  if (last_at + P > arena_cap) return -2;  // the sort pads the set to a power of two
  s.w.cur = arena + last_at;
  return finish_chart(s, dst, dst_cap, m_new, kept, n_last, accepting, h);
}

}  // namespace fmt
