// The trie sweep of the mask fill: one CTA per job (a row whose mask must be computed).
//
// For its job the CTA answers, for every trie node, "is the Earley set reached by this node's bytes
// non-empty?" (Sections 3.3 and 4.1: a token is valid iff every Earley set along its bytes stays
// non-empty).  Sets are hash-consed per job (AutoDev): a transition (set, byte class) is computed
// once, and every other node that needs it reads it from the set's record.  The automaton (records,
// items, hash), the job's base chart, the grammar's hot tables and the mask row under construction
// live in the CTA's shared memory; only automata that outgrow it spill into the CTA's slice of
// global memory.
//
// The trie is explored breadth first over the ALIVE nodes only: the frontier of a depth is a list of
// (node, Earley set) pairs; a warp takes some consecutive entries, lays their children out side by
// side (nodes are numbered breadth first, so the children of a node are consecutive) and gives each
// lane one child: next set = transition(parent's set, child's byte).  A transition nobody has
// computed yet belongs to the lane that claims it first: a step along a literal it takes on the
// spot (thread_step); anything else it queues for the warps (SweepWarp), which take the queued
// transitions, one each, once the depth has been laid out.  A child whose transition is queued or
// claimed by somebody else goes on a retry list, settled right after.  Only __syncthreads()
// separates the phases: nothing waits on another CTA or spins, and jobs are handed out through an
// atomic ticket.
#pragma once
#include "chart_step.cuh"

namespace fmt {

constexpr int SW_WARPS = 16;
constexpr int SW_THREADS = SW_WARPS * 32;
constexpr uint32_t SW_CUR = 256;        // items of a set under construction per warp (fast mode, power of two)
constexpr uint32_t SW_HSET = 512;       // uniqueness hash slots per warp (fast mode)
constexpr uint32_t SW_QUEUE = 512;      // transitions queued for the warps per round
constexpr uint32_t SW_HASH = 4096;      // slots of the shared-memory hash of Earley sets
constexpr uint32_t SW_HASH_MAX = 2560;  // sets it may hold; later ones go to the CTA's overflow hash
constexpr uint32_t SW_FRONT_SM = 256;   // entries of each frontier list kept in shared memory
constexpr uint32_t SW_SMEM_BUDGET = 227u * 1024u;
constexpr uint32_t SW_CHART_SM = 4096;  // words of a base chart staged in shared memory

// control words in shared memory
enum : uint32_t {
  SC_N_STATES = 0,   // Earley sets of the job so far
  SC_ITEMS_TOP,      // top of the shared-memory item pool
  SC_F_N0,           // entries of the frontier lists: three counters used in turn (depth mod 3), so that
  SC_F_N1,           // the one needed two depths ahead can be cleared while the other two are in use
  SC_F_N2,
  SC_RETRY_N0,       // entries of the retry list (two counters, by depth parity)
  SC_RETRY_N1,
  SC_FAIL,           // a capacity was exceeded: the row's mask cannot be trusted
  SC_GL_HASH,        // the overflow hash is in use
  SC_N_SMHASH,       // sets entered into the shared-memory hash
  SC_TRANS,          // transitions computed (statistics)
  SC_JOB,            // the job in hand
  SC_BIG,            // warps that switched to their large scratch (statistics)
  SC_Q_N,            // transitions queued for the warps
  SC_AGAIN,          // some node still waits after this round
  SC_TOTAL = 16
};

// word offsets into the dynamic shared memory
struct SweepSmem {
  uint32_t tables, mask, warps, warp_words, chart, hash, front, queue, ctl, recs, items, total;
};

__host__ __device__ inline uint32_t sw_pad4(uint32_t words) { return (words + 3u) & ~3u; }

__host__ __device__ inline SweepSmem sweep_smem(const GrammarDev& G, const AutoDev& A) {
  SweepSmem L;
  uint32_t at = 0;
  L.tables = at, at += sw_pad4(A.tables_in_smem ? G.hot_words : 0u);
  L.mask = at, at += sw_pad4(A.mask_in_smem ? G.Wm : 0u);
  L.warp_words = SW_CUR + SW_HSET + ((2u * G.Nw + 7u) & ~7u) + W_CTRS + 8u;
  L.warps = at, at += SW_WARPS * L.warp_words;
  L.chart = at, at += sw_pad4(A.chart_sm_words);
  L.hash = at, at += SW_HASH;
  L.front = at, at += 3u * 2u * SW_FRONT_SM;  // three lists of (node, set) pairs
  L.queue = at, at += SW_QUEUE;
  L.ctl = at, at += SC_TOTAL;
  L.recs = at, at += sw_pad4(A.sm_states * A.rec_words);
  L.items = at, at += sw_pad4(A.sm_items);
  L.total = at;
  return L;
}

__device__ __forceinline__ uint32_t ld_acquire_cta(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.cta.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t ld_volatile(const uint32_t* p) { return *reinterpret_cast<const volatile uint32_t*>(p); }

// What the CTA knows about its job and where the job's automaton lives.
struct CtaAuto {
  uint32_t rec_words, sm_states, sm_items, cap;
  uint32_t* ctl;       // shared
  uint32_t* sm_recs;   // shared
  uint32_t* sm_itm;    // shared
  uint32_t* sm_hash;   // shared
  uint32_t* gl_recs;   // this CTA's slice
  uint32_t* gl_hash;   // this CTA's slice
  uint32_t gl_hash_mask;
  uint32_t* gl_items;  // pool shared by all CTAs
  const uint32_t* base_off;
  const uint32_t* base_items;
  uint32_t m;          // live sets of the base chart

  __device__ __forceinline__ uint32_t* rec(uint32_t id) const {
    return id < sm_states ? sm_recs + id * rec_words : gl_recs + (size_t)(id - sm_states) * rec_words;
  }
  __device__ __forceinline__ uint32_t* items_at(uint32_t off) const {
    return off < sm_items ? sm_itm + off : gl_items + (off - sm_items);
  }
  __device__ __forceinline__ uint16_t* trans(uint32_t id) const { return reinterpret_cast<uint16_t*>(rec(id) + AR_TRANS); }
};

struct CtaView {
  const CtaAuto& a;
  __device__ __forceinline__ void operator()(uint32_t o, const uint32_t*& p, uint32_t& n) const {
    if (o < a.m) {
      const uint32_t x = a.base_off[o], y = a.base_off[o + 1];
      p = a.base_items + x;
      n = y - x;
    } else {
      const uint32_t* r = a.rec(o - a.m);
      p = a.items_at(r[AR_ITEMS]);
      n = r[AR_N];
    }
  }
  // an item of local state o that names its own state as origin means "origin o"
  __device__ __forceinline__ uint32_t fix(uint32_t item, uint32_t o) const {
    return ((item >> 16) == ORIGIN_SELF) ? ((o << 16) | (item & 0xFFFFu)) : item;
  }
};

// The Earley step of one warp.  Two forms of the same step (Section 3.2: scan, complete to a
// fixpoint, predict): while the scanned and completed items ("kernel") number at most 32 they sit
// one per lane and uniqueness is a matter of shuffles and ballots; larger sets go through the
// hash-based primitives of earley_device.cuh.  Either way the predicted items are a function of
// the kernel, so a set is looked up by its kernel alone (an order-independent hash, then an exact
// comparison as sets) BEFORE anything is predicted, and a set already known costs no prediction.
// A set's items are stored kernel first; nothing is sorted.
constexpr uint32_t T_RETRY = 0xfffffffbu;  // the lane-resident form does not apply: take the general one

struct SweepWarp {
  const GrammarDev& G;
  const StateDev& S;
  const CtaAuto& a;
  WarpCtx w;
  uint32_t* tmp8;     // shared
  uint32_t chunk_at = 0, chunk_left = 0;  // this warp's piece of the global item pool (lane 0's copy counts)

  // A new set with the items w.cur[0..n), the first nk of them its kernel: returns its id or T_FAIL.
  __device__ uint32_t create_set(uint32_t n, uint32_t nk, uint32_t hash) {
    const uint32_t lane = lane_id();
    uint32_t id = T_FAIL, ioff = 0;
    if (lane == 0) {
      const uint32_t got = atomicAdd(&a.ctl[SC_N_STATES], 1u);
      const uint32_t need = max(n, 1u);
      if (got < a.cap) {
        const uint32_t at = (ld_volatile(&a.ctl[SC_ITEMS_TOP]) < a.sm_items) ? atomicAdd(&a.ctl[SC_ITEMS_TOP], need) : a.sm_items;
        if (at < a.sm_items && need <= a.sm_items - at) {
          ioff = at;
          id = got;
        } else {
          if (need > chunk_left) {  // a new piece of the global pool: one atomic per ~4 Ki item words
            const uint32_t take = max(need, 4096u);
            chunk_at = atomicAdd(&S.counters[CNT_AUTO_ITEMS], take);
            chunk_left = (chunk_at <= S.au.items_cap && take <= S.au.items_cap - chunk_at) ? take : 0u;
          }
          if (need <= chunk_left) {
            ioff = a.sm_items + chunk_at;
            chunk_at += need;
            chunk_left -= need;
            id = got;
          }
        }
      }
    }
    id = __shfl_sync(FULL, id, 0);
    ioff = __shfl_sync(FULL, ioff, 0);
    if (id == T_FAIL) return T_FAIL;
    uint32_t* rec = a.rec(id);
    uint32_t* items = a.items_at(ioff);
    for (uint32_t i = lane; i < n; i += 32) items[i] = w.cur[i];
    for (uint32_t i = lane; i < a.rec_words; i += 32) {
      uint32_t v = 0u;
      if (i == AR_ITEMS) v = ioff;
      else if (i == AR_N) v = n;
      else if (i == AR_HASH) v = hash;
      else if (i == AR_NK) v = nk;
      else if (i >= AR_SCAN && i < AR_SCAN + 8) v = tmp8[i - AR_SCAN];
      else if (i >= AR_TRANS) v = 0xFFFFFFFFu;  // two T16_UNKNOWN
      rec[i] = v;
    }
    __syncwarp();
    __threadfence_block();
    return id;
  }

  // The set whose kernel has nk items and this hash and consists of items for which `member`
  // holds: its id, or T_FAIL if there is none.  member(x, valid) is called by all lanes.
  template <class Member>
  __device__ uint32_t lookup_set(uint32_t nk, uint32_t hash, Member member) {
    const uint32_t lane = lane_id();
    for (int t = 0; t < 2; ++t) {
      if (t == 1 && !ld_volatile(&a.ctl[SC_GL_HASH])) break;
      const uint32_t* table = t ? a.gl_hash : a.sm_hash;
      const uint32_t mask = t ? a.gl_hash_mask : SW_HASH - 1u;
      uint32_t slot = hash & mask;
      for (uint32_t probe = 0; probe <= mask; ++probe) {
        uint32_t v = 0;
        if (lane == 0) v = ld_acquire_cta(&table[slot]);
        v = __shfl_sync(FULL, v, 0);
        if (v == 0) break;
        if (same_set(v - 1u, nk, hash, member)) return v - 1u;
        slot = (slot + 1u) & mask;
      }
    }
    return T_FAIL;
  }

  // Is the set `sid` the one with this hash and a kernel of nk items for which `member` holds?
  template <class Member>
  __device__ __forceinline__ bool same_set(uint32_t sid, uint32_t nk, uint32_t hash, Member member) {
    const uint32_t lane = lane_id();
    const uint32_t* rec = a.rec(sid);
    if (ld_volatile(rec + AR_HASH) != hash || ld_volatile(rec + AR_NK) != nk) return false;
    const uint32_t* items = a.items_at(ld_volatile(rec + AR_ITEMS));
    bool ok = true;
    for (uint32_t base = 0; base < nk; base += 32) {
      const bool valid = base + lane < nk;
      const uint32_t x = valid ? ld_volatile(items + base + lane) : 0u;
      ok = member(x, valid) && ok;
    }
    return __all_sync(FULL, ok);
  }

  // Enter the freshly created set `id` into the hash, unless an equal set got there first (several
  // warps often reach the same new set at the same moment): returns the id to use.
  template <class Member>
  __device__ uint32_t insert_set(uint32_t id, uint32_t nk, uint32_t hash, Member member) {
    const uint32_t lane = lane_id();
    uint32_t use_gl = 0;
    if (lane == 0) {
      use_gl = ld_volatile(&a.ctl[SC_GL_HASH]);
      if (!use_gl && atomicAdd(&a.ctl[SC_N_SMHASH], 1u) >= SW_HASH_MAX) {
        atomicExch(&a.ctl[SC_GL_HASH], 1u);
        use_gl = 1u;
      }
    }
    use_gl = __shfl_sync(FULL, use_gl, 0);
    uint32_t* table = use_gl ? a.gl_hash : a.sm_hash;
    const uint32_t mask = use_gl ? a.gl_hash_mask : SW_HASH - 1u;
    uint32_t slot = hash & mask;
    for (uint32_t probe = 0; probe <= mask; ++probe) {
      uint32_t old = 0;
      if (lane == 0) old = atomicCAS(&table[slot], 0u, id + 1u);
      old = __shfl_sync(FULL, old, 0);
      if (old == 0u) return id;
      __threadfence_block();
      if (same_set(old - 1u, nk, hash, member)) return old - 1u;
      slot = (slot + 1u) & mask;
    }
    return T_FAIL;
  }

  // The kernel w.cur[0..nk) is new: predict, describe, store and enter the set.
  template <class Member>
  __device__ uint32_t finish_new(uint32_t nk, uint32_t hash, Member member) {
    const uint32_t lane = lane_id();
    __syncwarp();
    if (lane == 0) w.ctr[W_NCUR] = nk, w.ctr[W_OVERFLOW] = 0u;
    predict_into_cur(G, w, ORIGIN_SELF);
    if (w.ctr[W_OVERFLOW]) return T_RETRY;
    const uint32_t n = min(w.ctr[W_NCUR], w.cur_cap);
    scannable_bytes(G, w.cur, n, tmp8);
    const uint32_t id = create_set(n, nk, hash);
    return id == T_FAIL ? T_FAIL : insert_set(id, nk, hash, member);
  }

  // (lane-resident form) The candidates c .. c + skip of the lanes with `v` set join cur[0..n)
  // unless already there.  `mine` is cur[lane].  Returns the new count, above 32 when they do not fit.
  __device__ __forceinline__ uint32_t append_small(uint32_t c, bool v, uint32_t skip, uint32_t n, uint32_t& mine) {
    const uint32_t lane = lane_id();
    const uint32_t maxskip = __reduce_max_sync(FULL, v ? skip : 0u);
    for (uint32_t j = 0; j <= maxskip; ++j) {
      const bool vj = v && j <= skip;
      const uint32_t cj = c + j;
      const uint32_t vm = __ballot_sync(FULL, vj);
      if (!vm) continue;
      bool keep = vj;
      if (vj) keep = (uint32_t)(__ffs(__match_any_sync(vm, cj)) - 1) == lane;  // one of equal candidates
      for (uint32_t i = 0; i < n; ++i)
        if (__shfl_sync(FULL, mine, i) == cj) keep = false;
      const uint32_t kb = __ballot_sync(FULL, keep);
      const uint32_t nn = n + __popc(kb);
      if (nn > 32u) return nn;
      if (keep) w.cur[n + __popc(kb & ((1u << lane) - 1u))] = cj;
      __syncwarp();
      n = nn;
      mine = lane < n ? w.cur[lane] : 0u;
    }
    return n;
  }

  __device__ uint32_t compute_small(uint32_t ps, uint32_t byte) {
    const uint32_t lane = lane_id();
    const uint32_t* pitems;
    uint32_t plen;
    CtaView view{a};
    view(ps == 0 ? a.m - 1 : a.m + ps, pitems, plen);
    const uint32_t self_code = a.m + ps;
    uint32_t n = 0, mine = 0;
    __syncwarp();
    // ---- scan
    for (uint32_t base = 0; base < plen; base += 32) {
      const uint32_t k = base + lane;
      uint32_t it = k < plen ? pitems[k] : 0u;
      const uint32_t inf = k < plen ? G.info[it & 0xFFFFu] : 0u;
      const bool hit = (inf >> INFO_KIND_SHIFT) == KIND_TERM && class_has(G, inf & INFO_ARG_MASK, byte);
      if ((it >> 16) == ORIGIN_SELF) it = (self_code << 16) | (it & 0xFFFFu);
      const uint32_t skip = hit ? (G.info[(it + 1u) & 0xFFFFu] >> INFO_SKIP_SHIFT) & INFO_SKIP_MASK : 0u;
      if (__any_sync(FULL, hit)) n = append_small(it + 1u, hit, skip, n, mine);
      if (n > 32u) return T_RETRY;
    }
    if (n == 0) return T_DEAD;
    // ---- complete to a fixpoint: lanes [head, n) hold the items not looked at yet
    uint32_t head = 0;
    while (head < n) {
      const bool have = lane >= head && lane < n;
      const uint32_t inf = have ? G.info[mine & 0xFFFFu] : 0u;
      const uint32_t kind = inf >> INFO_KIND_SHIFT;
      if (have && kind == KIND_NT) {
        const uint32_t y = inf & INFO_ARG_MASK;
        atomicOr(&w.nt[y >> 5], 1u << (y & 31u));
      }
      uint32_t bal = __ballot_sync(FULL, have && kind == KIND_END && (mine >> 16) != ORIGIN_SELF);
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
            return T_RETRY;
          }
        }
      }
    }
    // ---- the kernel: what is left when the completed items go
    const bool keep = lane < n && (G.info[mine & 0xFFFFu] >> INFO_KIND_SHIFT) != KIND_END;
    const uint32_t kb = __ballot_sync(FULL, keep);
    const uint32_t nk = __popc(kb);
    uint32_t h = keep ? mix32(mine) : 0u;
    for (int d = 16; d > 0; d >>= 1) h += __shfl_xor_sync(FULL, h, d);
    h = mix32(h + nk * 0x9E3779B9u);
    __syncwarp();
    if (keep) w.cur[__popc(kb & ((1u << lane) - 1u))] = mine;
    __syncwarp();
    mine = lane < nk ? w.cur[lane] : 0u;
    auto member = [&](uint32_t x, bool valid) {  // the kernel sits one item per lane
      bool found = false;
      for (uint32_t i = 0; i < nk; ++i)
        if (__shfl_sync(FULL, mine, i) == x) found = true;
      return found || !valid;
    };
    const uint32_t id = lookup_set(nk, h, member);
    if (id != T_FAIL) {
      clear_nt(G, w);
      return id;
    }
    return finish_new(nk, h, member);
  }

  // The general form, for sets of any size (w.cur may be the warp's large area).
  __device__ uint32_t compute_general(uint32_t ps, uint32_t byte) {
    const uint32_t lane = lane_id();
    const uint32_t* pitems;
    uint32_t plen;
    CtaView view{a};
    view(ps == 0 ? a.m - 1 : a.m + ps, pitems, plen);
    __syncwarp();
    if (lane < W_CTRS) w.ctr[lane] = 0u;
    __syncwarp();
    const uint32_t self_code = a.m + ps;
    for (uint32_t k = lane; k < plen; k += 32) {
      uint32_t it = pitems[k];
      uint32_t inf = G.info[it & 0xFFFFu];
      if ((inf >> INFO_KIND_SHIFT) == KIND_TERM && class_has(G, inf & INFO_ARG_MASK, byte)) {
        if ((it >> 16) == ORIGIN_SELF) it = (self_code << 16) | (it & 0xFFFFu);
        add_item(G, w, it + 1u);
      }
    }
    __syncwarp();
    if (w.ctr[W_OVERFLOW]) {
      hset_clear_all(w.hset, w.hset_mask);
      return T_FAIL;
    }
    if (w.ctr[W_NCUR] == 0u) return T_DEAD;
    complete_fixpoint(G, w, view, ORIGIN_SELF, 0u);
    const uint32_t hashed = min(w.ctr[W_NCUR], w.cur_cap);
    if (w.ctr[W_OVERFLOW]) {
      hset_clear_all(w.hset, w.hset_mask);
      clear_nt(G, w);
      return T_FAIL;
    }
    // the kernel: the items that are not completed; all of cur[0..hashed) are in the uniqueness hash
    uint32_t nk = 0, h = 0;
    for (uint32_t base = 0; base < hashed; base += 32) {
      const uint32_t i = base + lane;
      const uint32_t it = i < hashed ? w.cur[i] : 0u;
      const bool keep = i < hashed && (G.info[it & 0xFFFFu] >> INFO_KIND_SHIFT) != KIND_END;
      if (keep) h += mix32(it);
      nk += __popc(__ballot_sync(FULL, keep));
    }
    for (int d = 16; d > 0; d >>= 1) h += __shfl_xor_sync(FULL, h, d);
    h = mix32(h + nk * 0x9E3779B9u);
    const uint32_t id = lookup_set(nk, h, [&](uint32_t x, bool valid) { return !valid || hset_contains(w.hset, w.hset_mask, x); });
    hset_clear_items(w, hashed);
    if (id != T_FAIL) {
      clear_nt(G, w);
      return id;
    }
    drop_completed(G, w, hashed);
    // the kernel is cur[0..nk) now and no longer in the hash: a set met while entering this one is compared item by item
    const uint32_t r = finish_new(nk, h, [&](uint32_t x, bool valid) {
      bool found = !valid;
      for (uint32_t i = 0; i < nk && !found; ++i) found = w.cur[i] == x;
      return found;
    });
    return r == T_RETRY ? T_FAIL : r;
  }
};

// ---- the Earley step of one THREAD, for the commonest transition there is: along the bytes of a
// literal, where a set of a few items, each with a terminal after the dot, scans into a set of the
// same kind.  Nothing completes and nothing is predicted, so the new set is just the scanned
// items; the thread that claimed the transition computes it on the spot and its node needs no
// second visit.  Anything else (more than TS_MAX items, an item that ends or meets a non-terminal)
// is left to the warps.  Sets are entered with the same hash and the same compare-on-conflict
// protocol as the warps use, so both kinds of step find each other's sets.
constexpr uint32_t TS_MAX = 6;
constexpr uint32_t TS_WARP = 0xfffffffau;  // not a case for a single thread

__device__ __forceinline__ bool ts_same(const CtaAuto& a, uint32_t sid, const uint32_t (&out)[TS_MAX], uint32_t cnt, uint32_t h) {
  const uint32_t* rec = a.rec(sid);
  if (ld_volatile(rec + AR_HASH) != h || ld_volatile(rec + AR_NK) != cnt) return false;
  const uint32_t* items = a.items_at(ld_volatile(rec + AR_ITEMS));
  bool same = true;
#pragma unroll
  for (uint32_t i = 0; i < TS_MAX; ++i) {
    if (i < cnt) {
      const uint32_t x = ld_volatile(items + i);
      bool found = false;
#pragma unroll
      for (uint32_t k = 0; k < TS_MAX; ++k) found |= (k < cnt && out[k] == x);
      same &= found;
    }
  }
  return same;
}

__device__ uint32_t thread_step(const GrammarDev& G, const StateDev& S, const CtaAuto& a, uint32_t ps, uint32_t byte) {
  const uint32_t* pitems;
  uint32_t plen;
  CtaView view{a};
  view(ps == 0 ? a.m - 1 : a.m + ps, pitems, plen);
  if (plen > TS_MAX) return TS_WARP;
  const uint32_t self_code = a.m + ps;
  uint32_t out[TS_MAX];
  uint32_t scan[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) scan[i] = 0u;
  uint32_t cnt = 0, hsum = 0;
#pragma unroll
  for (uint32_t k = 0; k < TS_MAX; ++k) {
    out[k] = 0u;
    if (k < plen) {
      uint32_t it = pitems[k];
      const uint32_t inf = G.info[it & 0xFFFFu];
      if ((inf >> INFO_KIND_SHIFT) == KIND_TERM && class_has(G, inf & INFO_ARG_MASK, byte)) {
        if ((it >> 16) == ORIGIN_SELF) it = (self_code << 16) | (it & 0xFFFFu);
        const uint32_t c = it + 1u;
        const uint32_t cinf = G.info[c & 0xFFFFu];
        if ((cinf >> INFO_KIND_SHIFT) != KIND_TERM) return TS_WARP;
        const uint4* cb = reinterpret_cast<const uint4*>(G.class_bits + (cinf & INFO_ARG_MASK) * 8u);
        const uint4 x = cb[0], y = cb[1];
        scan[0] |= x.x, scan[1] |= x.y, scan[2] |= x.z, scan[3] |= x.w;
        scan[4] |= y.x, scan[5] |= y.y, scan[6] |= y.z, scan[7] |= y.w;
#pragma unroll
        for (uint32_t q = 0; q < TS_MAX; ++q)
          if (q == cnt) out[q] = c;
        ++cnt;
        hsum += mix32(c);
      }
    }
  }
  if (cnt == 0) return T_DEAD;
  const uint32_t h = mix32(hsum + cnt * 0x9E3779B9u);
  // ---- known already?
  for (int t = 0; t < 2; ++t) {
    if (t == 1 && !ld_volatile(&a.ctl[SC_GL_HASH])) break;
    const uint32_t* table = t ? a.gl_hash : a.sm_hash;
    const uint32_t mask = t ? a.gl_hash_mask : SW_HASH - 1u;
    uint32_t slot = h & mask;
    for (uint32_t probe = 0; probe <= mask; ++probe) {
      const uint32_t v = ld_acquire_cta(&table[slot]);
      if (v == 0) break;
      if (ts_same(a, v - 1u, out, cnt, h)) return v - 1u;
      slot = (slot + 1u) & mask;
    }
  }
  // ---- a new set
  const uint32_t id = atomicAdd(&a.ctl[SC_N_STATES], 1u);
  if (id >= a.cap) return T_FAIL;
  uint32_t ioff;
  {
    const uint32_t at = (ld_volatile(&a.ctl[SC_ITEMS_TOP]) < a.sm_items) ? atomicAdd(&a.ctl[SC_ITEMS_TOP], cnt) : a.sm_items;
    if (at < a.sm_items && cnt <= a.sm_items - at) {
      ioff = at;
    } else {
      const uint32_t g = atomicAdd(&S.counters[CNT_AUTO_ITEMS], cnt);
      if (g > S.au.items_cap || cnt > S.au.items_cap - g) return T_FAIL;
      ioff = a.sm_items + g;
    }
  }
  uint32_t* items = a.items_at(ioff);
#pragma unroll
  for (uint32_t i = 0; i < TS_MAX; ++i)
    if (i < cnt) items[i] = out[i];
  uint32_t* rec = a.rec(id);
  rec[AR_ITEMS] = ioff, rec[AR_N] = cnt, rec[AR_HASH] = h, rec[AR_NK] = cnt;
#pragma unroll
  for (int i = 0; i < 8; ++i) rec[AR_SCAN + i] = scan[i];
  for (uint32_t i = AR_TRANS; i < a.rec_words; ++i) rec[i] = 0xFFFFFFFFu;
  __threadfence_block();
  uint32_t use_gl = ld_volatile(&a.ctl[SC_GL_HASH]);
  if (!use_gl && atomicAdd(&a.ctl[SC_N_SMHASH], 1u) >= SW_HASH_MAX) {
    atomicExch(&a.ctl[SC_GL_HASH], 1u);
    use_gl = 1u;
  }
  uint32_t* table = use_gl ? a.gl_hash : a.sm_hash;
  const uint32_t mask = use_gl ? a.gl_hash_mask : SW_HASH - 1u;
  uint32_t slot = h & mask;
  for (uint32_t probe = 0; probe <= mask; ++probe) {
    const uint32_t old = atomicCAS(&table[slot], 0u, id + 1u);
    if (old == 0u) return id;
    __threadfence_block();
    if (ts_same(a, old - 1u, out, cnt, h)) return old - 1u;
    slot = (slot + 1u) & mask;
  }
  return T_FAIL;
}

__device__ __forceinline__ void set_tokens(const GrammarDev& G, uint32_t* mask, uint32_t node) {
  const uint32_t tok = __ldg(&G.node_tok[node]);
  if (tok == NODE_TOK_NONE) return;
  if (tok != NODE_TOK_MANY) {
    atomicOr(&mask[tok >> 5], 1u << (tok & 31u));
    return;
  }
  for (uint32_t i = __ldg(&G.tok_off[node]), e = __ldg(&G.tok_off[node + 1]); i < e; ++i) {
    const uint32_t t = __ldg(&G.tok_ids[i]);
    atomicOr(&mask[t >> 5], 1u << (t & 31u));
  }
}

constexpr uint32_t ST_WAIT = 0xFFFEu;  // the transition is not known yet: the node goes on the retry list

// The set a node reaches from its parent's set `ps` on `byte`: ST_DEAD, ST_WAIT or the set's id.  An
// unknown transition is claimed: the claimer takes a step along a literal itself, here and now, and
// queues anything else for the warps.
__device__ __forceinline__ uint32_t step_node(const GrammarDev& G, const StateDev& S, const CtaAuto& a, uint32_t* queue,
                                              uint32_t ps, uint32_t byte) {
  const uint32_t* rec = a.rec(ps);
  // one 256-bit test rejects most bytes without touching the transition table
  if (!((rec[AR_SCAN + (byte >> 5)] >> (byte & 31u)) & 1u)) return ST_DEAD;
  uint16_t* tr = a.trans(ps) + G.eq_of_byte[byte];
  uint32_t t = *reinterpret_cast<volatile uint16_t*>(tr);
  if (t == T16_UNKNOWN) {
    t = atomicCAS(tr, (unsigned short)T16_UNKNOWN, (unsigned short)T16_PENDING);
    if (t == T16_UNKNOWN) {  // ours
      uint32_t r = thread_step(G, S, a, ps, byte);
      if (r != TS_WARP) {
        if (r == T_FAIL) a.ctl[SC_FAIL] = 1u, r = T_DEAD;
        atomicAdd(&a.ctl[SC_TRANS], 1u);
        *reinterpret_cast<volatile uint16_t*>(tr) = (r == T_DEAD) ? T16_DEAD : (uint16_t)r;
        return (r == T_DEAD) ? (uint32_t)ST_DEAD : r;
      }
      const uint32_t at = atomicAdd(&a.ctl[SC_Q_N], 1u);
      if (at < SW_QUEUE) queue[at] = (ps << 8) | byte;
      else *reinterpret_cast<volatile uint16_t*>(tr) = T16_UNKNOWN;  // no room in this round: somebody claims it again in the next
      return ST_WAIT;
    }
  }
  if (t == T16_PENDING || t == T16_UNKNOWN) return ST_WAIT;
  return (t == T16_DEAD) ? (uint32_t)ST_DEAD : t;
}

// A list of (node, Earley set) pairs: the first SW_FRONT_SM entries in shared memory, the rest in the
// CTA's slice of global memory.
struct NodeList {
  uint2* sm;
  uint2* gl;
  __device__ __forceinline__ uint2 get(uint32_t i) const { return i < SW_FRONT_SM ? sm[i] : gl[i - SW_FRONT_SM]; }
  __device__ __forceinline__ void put(uint32_t i, uint2 v) const {
    if (i < SW_FRONT_SM) sm[i] = v;
    else gl[i - SW_FRONT_SM] = v;
  }
  // (all lanes) append the pairs of the lanes with `v` set
  __device__ __forceinline__ void push(uint32_t* counter, bool v, uint32_t node, uint32_t set) const {
    const uint32_t bal = __ballot_sync(FULL, v);
    if (!bal) return;
    const uint32_t lane = lane_id();
    uint32_t at = 0;
    if (lane == 0) at = atomicAdd(counter, (uint32_t)__popc(bal));
    at = __shfl_sync(FULL, at, 0);
    if (v) put(at + __popc(bal & ((1u << lane) - 1u)), make_uint2(node, set));
  }
};

__global__ void __launch_bounds__(SW_THREADS, 1) sweep_kernel(GrammarDev Gg, StateDev S) {
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  if (blockIdx.x >= n_jobs) return;  // more CTAs than jobs
  extern __shared__ __align__(16) uint32_t smem[];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = lane_id();
  const AutoDev& A = S.au;
  const SweepSmem L = sweep_smem(Gg, A);
  GrammarDev G = Gg;
  if (A.tables_in_smem) G = stage_hot_tables(Gg, smem + L.tables);
  uint32_t* const ctl = smem + L.ctl;
  uint32_t* const queue = smem + L.queue;
  uint32_t* const chart_sm = smem + L.chart;
  uint32_t* const mask_sm = smem + L.mask;

  CtaAuto a;
  a.rec_words = A.rec_words, a.sm_states = A.sm_states, a.sm_items = A.sm_items;
  a.ctl = ctl;
  a.sm_recs = smem + L.recs;
  a.sm_itm = smem + L.items;
  a.sm_hash = smem + L.hash;
  a.gl_recs = A.recs + (size_t)blockIdx.x * (A.cap - A.sm_states) * A.rec_words;
  a.gl_hash = A.hash + (size_t)blockIdx.x * (A.gl_hash_mask + 1u);
  a.gl_hash_mask = A.gl_hash_mask;
  a.gl_items = A.items;
  // two frontiers (used by depth parity) and the retry list
  uint2* const front_sm = reinterpret_cast<uint2*>(smem + L.front);
  uint2* const front_gl = A.front + (size_t)blockIdx.x * 3u * A.level_pad;
  const NodeList list_even{front_sm, front_gl}, list_odd{front_sm + SW_FRONT_SM, front_gl + A.level_pad};
  const NodeList retry{front_sm + 2u * SW_FRONT_SM, front_gl + 2u * (size_t)A.level_pad};

  uint32_t* mine = smem + L.warps + (size_t)warp * L.warp_words;
  SweepWarp sw{G, S, a};
  sw.w.cur = mine;
  sw.w.cur_cap = SW_CUR;
  sw.w.hset = mine + SW_CUR;
  sw.w.hset_mask = SW_HSET - 1;
  sw.w.nt = sw.w.hset + SW_HSET;
  const uint32_t ntw = (2u * G.Nw + 7u) & ~7u;
  sw.w.ctr = sw.w.nt + ntw;
  sw.tmp8 = sw.w.ctr + W_CTRS;
  uint32_t* const big = S.big_scratch + ((size_t)blockIdx.x * SW_WARPS + warp) * ((size_t)S.big_arena_items + S.big_hset_slots);
  bool big_mode = false;
  hset_clear_all(sw.w.hset, SW_HSET - 1);
  for (uint32_t i = lane; i < ntw; i += 32) sw.w.nt[i] = 0u;
  if (tid < SC_TOTAL) ctl[tid] = 0u;
  uint32_t stat_trans = 0, stat_states = 0;  // thread 0's copies count

  // (all lanes) the transition of set ps on byte pb, by the whole warp
  auto warp_transition = [&](uint32_t ps, uint32_t pb) -> uint32_t {
    uint32_t r = big_mode ? T_RETRY : sw.compute_small(ps, pb);
    if (r == T_RETRY) r = sw.compute_general(ps, pb);
    if (r == T_FAIL && !big_mode) {  // a set outgrew the shared-memory scratch: use the large area from now on
      big_mode = true;
      hset_clear_all(sw.w.hset, sw.w.hset_mask);
      clear_nt(G, sw.w);
      sw.w.cur = big;
      sw.w.cur_cap = S.big_arena_items;
      sw.w.hset = big + S.big_arena_items;
      sw.w.hset_mask = S.big_hset_slots - 1;
      if (lane == 0) atomicAdd(&ctl[SC_BIG], 1u);
      r = sw.compute_general(ps, pb);
    }
    if (r == T_FAIL) {  // a capacity was exceeded: the row's mask cannot be trusted
      hset_clear_all(sw.w.hset, sw.w.hset_mask);
      clear_nt(G, sw.w);
      if (lane == 0) ctl[SC_FAIL] = 1u;
      r = T_DEAD;  // lets the sweep go on
    }
    return r;
  };

  for (;;) {
    __syncthreads();
    const bool gl_hash_dirty = ctl[SC_GL_HASH] != 0u;  // left by the job before
    __syncthreads();
    if (tid == 0) ctl[SC_JOB] = atomicAdd(&S.counters[CNT_JOB_NEXT], 1u);
    __syncthreads();
    const uint32_t j = ctl[SC_JOB];
    if (j >= n_jobs) {  // leave the overflow hash all zero for the next launch
      if (gl_hash_dirty)
        for (uint32_t i = tid; i <= a.gl_hash_mask; i += SW_THREADS) a.gl_hash[i] = 0u;
      break;
    }

    // ---- the job: its chart, an automaton with one state (the chart's last set), an empty mask
    const uint32_t row = S.jobs[j];
    const uint32_t* chart = S.arena + S.row_chart[row];
    const uint32_t m = chart[CH_SETS];
    const uint32_t chart_words = chart[CH_WORDS];
    const bool accepting = (chart[CH_FLAGS] & CHART_ACCEPTING) != 0u;
    uint32_t* const mask = A.mask_in_smem ? mask_sm : S.mask_rows + (size_t)S.row_mask[row] * G.Wm;
    if (chart_words <= A.chart_sm_words) {
      for (uint32_t i = tid; i < chart_words; i += SW_THREADS) chart_sm[i] = chart[i];
      chart = chart_sm;
    }
    a.base_off = chart + CH_HDR;
    a.base_items = chart + CH_HDR + m + 1;
    a.m = m;
    a.cap = min(min(A.cap, AUTO_MAX_STATES), (ORIGIN_SELF - 1u > m) ? ORIGIN_SELF - 1u - m : 0u);
    for (uint32_t i = tid; i < SW_HASH; i += SW_THREADS) a.sm_hash[i] = 0u;
    if (gl_hash_dirty)
      for (uint32_t i = tid; i <= a.gl_hash_mask; i += SW_THREADS) a.gl_hash[i] = 0u;
    for (uint32_t i = tid; i < G.Wm; i += SW_THREADS) mask[i] = 0u;
    if (tid < SC_TOTAL && tid != SC_JOB) ctl[tid] = 0u;
    uint32_t* rec0 = a.rec(0);
    for (uint32_t i = tid; i < a.rec_words; i += SW_THREADS)
      if (i < AR_SCAN || i >= AR_SCAN + 8) rec0[i] = (i >= AR_TRANS) ? 0xFFFFFFFFu : 0u;
    __syncthreads();
    if (warp == 0) {
      scannable_bytes(G, a.base_items + a.base_off[m - 1], a.base_off[m] - a.base_off[m - 1], sw.tmp8);
      if (lane < 8) rec0[AR_SCAN + lane] = sw.tmp8[lane];
      if (lane == 0) {
        ctl[SC_N_STATES] = 1u;
        list_even.put(0, make_uint2(0u, 0u));  // depth 0: the root, in state 0
        ctl[SC_F_N0] = 1u;
        if (accepting && G.eos >= 0) mask[(uint32_t)G.eos >> 5] = 1u << ((uint32_t)G.eos & 31u);
      }
    }
    __syncthreads();

    for (uint32_t Lv = 0; Lv <= G.depth; ++Lv) {
      const uint32_t F = ctl[SC_F_N0 + Lv % 3u];  // nodes of depth Lv that are alive
      if (F == 0) break;
      uint32_t* const next_n = &ctl[SC_F_N0 + (Lv + 1u) % 3u];
      uint32_t* const retry_n = &ctl[SC_RETRY_N0 + (Lv & 1u)];
      if (tid == 0) ctl[SC_F_N0 + (Lv + 2u) % 3u] = 0u, ctl[SC_RETRY_N0 + ((Lv + 1u) & 1u)] = 0u;  // for the next depth
      const NodeList cur = (Lv & 1u) ? list_odd : list_even, next = (Lv & 1u) ? list_even : list_odd;
      // a warp takes `grp` consecutive entries at a time: one when there are few, so that their
      // transitions are computed by different warps
      const uint32_t grp = (F <= (uint32_t)SW_WARPS) ? 1u : min(32u, (F + 2u * SW_WARPS - 1u) / (2u * SW_WARPS));
      for (uint32_t p0 = warp * grp; p0 < F; p0 += SW_WARPS * grp) {
        const uint32_t np = min(grp, F - p0);
        uint32_t pst = ST_DEAD, c0 = 0, cnt = 0;
        if (lane < np) {
          const uint2 e = cur.get(p0 + lane);
          pst = e.y;
          c0 = __ldg(&G.child_off[e.x]);
          cnt = __ldg(&G.child_off[e.x + 1u]) - c0;
          if (e.x != 0u) set_tokens(G, mask, e.x);  // the node is alive: so are the tokens that end there
        }
        uint32_t incl = cnt;
        for (int d = 1; d < 32; d <<= 1) {
          const uint32_t t = __shfl_up_sync(FULL, incl, d);
          if ((int)lane >= d) incl += t;
        }
        const uint32_t total = __shfl_sync(FULL, incl, 31);
        for (uint32_t base = 0; base < total; base += 32) {
          const uint32_t idx = base + lane;
          const bool valid = idx < total;
          uint32_t p = 0;  // the parent whose children include the idx-th child: how many prefix sums are <= idx
#pragma unroll
          for (uint32_t sft = 16; sft > 0; sft >>= 1) {
            const uint32_t v = __shfl_sync(FULL, incl, (p + sft - 1u) & 31u);
            if (v <= idx && p + sft <= 32u) p += sft;
          }
          p &= 31u;
          const uint32_t p_incl = __shfl_sync(FULL, incl, p), p_cnt = __shfl_sync(FULL, cnt, p);
          const uint32_t p_c0 = __shfl_sync(FULL, c0, p), ps = __shfl_sync(FULL, pst, p);
          const uint32_t child = p_c0 + (idx - (p_incl - p_cnt));
          const uint32_t byte = valid ? __ldg(&G.node_byte[child]) : 0u;
          const uint32_t t = valid ? step_node(G, S, a, queue, ps, byte) : (uint32_t)ST_DEAD;
          next.push(next_n, valid && t != ST_DEAD && t != ST_WAIT, child, t);
          retry.push(retry_n, t == ST_WAIT, child, ps);
        }
      }
      __syncthreads();
      // ---- the warps compute the queued transitions, then the children that waited are settled;
      // again while some still wait (only when more transitions were queued than the queue holds)
      const uint32_t R = *retry_n;
      for (uint32_t rounds = 0;; ++rounds) {
        const uint32_t nq = min(ctl[SC_Q_N], SW_QUEUE);
        if (nq == 0 && !(rounds == 0 ? R > 0 : ctl[SC_AGAIN] != 0u)) break;
        if (rounds > (1u << 16)) {  // cannot happen (every round settles at least one transition); never spin
          if (tid == 0) ctl[SC_FAIL] = 1u;
          break;
        }
        for (uint32_t i = warp; i < nq; i += SW_WARPS) {
          const uint32_t ps = queue[i] >> 8, pb = queue[i] & 0xFFu;
          const uint32_t r = warp_transition(ps, pb);
          if (lane == 0) {
            *reinterpret_cast<volatile uint16_t*>(a.trans(ps) + G.eq_of_byte[pb]) = (r == T_DEAD) ? T16_DEAD : (uint16_t)r;
            atomicAdd(&ctl[SC_TRANS], 1u);
          }
        }
        __syncthreads();
        if (tid == 0) ctl[SC_Q_N] = 0u, ctl[SC_AGAIN] = 0u;
        __syncthreads();
        for (uint32_t base = 0; base < R; base += SW_THREADS) {
          const uint32_t i = base + tid;
          uint32_t child = 0xFFFFFFFFu, t = ST_DEAD;
          if (i < R) {
            const uint2 e = retry.get(i);
            child = e.x;
            if (child != 0xFFFFFFFFu) {  // not settled in an earlier round
              t = step_node(G, S, a, queue, e.y, __ldg(&G.node_byte[child]));
              if (t == ST_WAIT) ctl[SC_AGAIN] = 1u;
              else retry.put(i, make_uint2(0xFFFFFFFFu, 0u));
            }
          }
          next.push(next_n, t != ST_DEAD && t != ST_WAIT, child, t);
        }
        __syncthreads();
      }
      __syncthreads();  // everybody has seen this depth's counters before the next depth changes them
    }

    // ---- the job's result
    __syncthreads();
    const bool failed = ctl[SC_FAIL] != 0u;
    if (A.mask_in_smem) {
      uint32_t* out = S.mask_rows + (size_t)S.row_mask[row] * G.Wm;
      for (uint32_t i = tid; i < G.Wm; i += SW_THREADS) out[i] = mask_sm[i];
    }
    if (tid == 0) {
      if (failed) {
        atomicOr(&S.row_flags[row], ROW_BROKEN);
        atomicExch(&S.counters[CNT_ERR], 1u);
        stat_add(S, CNT_STAT_CAPERR, 1u);
      }
      stat_trans += ctl[SC_TRANS];
      stat_states += min(ctl[SC_N_STATES], a.cap) - 1u;
      if (ctl[SC_BIG]) stat_add(S, CNT_STAT_BIG, ctl[SC_BIG]);
    }
  }
  if (big_mode) hset_clear_all(sw.w.hset, sw.w.hset_mask);
  if (tid == 0) {
    stat_add(S, CNT_STAT_TRANS, stat_trans);
    stat_add(S, CNT_STAT_LOCAL, stat_states);
  }
}

}  // namespace fmt
