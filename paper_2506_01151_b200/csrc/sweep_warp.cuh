// Device code shared by the trie sweep and the context-dependent walk: one warp computing one Earley
// step (Section 3.2: scan, complete to a fixpoint, predict) of an automaton of hash-consed Earley sets.
#pragma once
#include "earley_device.cuh"

namespace fmt {

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned long long ld_acquire64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint64_t ld_cg64(const uint64_t* p) {
  return (uint64_t)__ldcg(reinterpret_cast<const unsigned long long*>(p));
}
__device__ __forceinline__ void stat_add(const StateDev& S, uint32_t slot, uint32_t v) {
  atomicAdd(reinterpret_cast<unsigned long long*>(S.counters + slot), (unsigned long long)v);
}
__device__ __forceinline__ void stat_add64(const StateDev& S, uint32_t slot, unsigned long long v) {
  atomicAdd(reinterpret_cast<unsigned long long*>(S.counters + slot), v);
}
__device__ __forceinline__ void diag(const StateDev& S, uint32_t what) { atomicAdd(S.counters + CNT_DIAG + what, 1u); }
__device__ __forceinline__ void stat_max(const StateDev& S, uint32_t slot, uint32_t v) { atomicMax(S.counters + slot, v); }

constexpr uint32_t HOT_TABLE_BYTES = 24 * 1024;  // grammar tables up to this size are staged in shared memory

constexpr uint32_t SWEEP_CUR = 512;     // items of a set under construction per warp (fast mode, power of two)
constexpr uint32_t SWEEP_HSET = 1024;   // uniqueness hash slots per warp (fast mode)

struct JobCtx {
  const uint32_t* base_off;
  const uint32_t* base_items;
  uint32_t m;         // live sets of the base chart
  uint32_t* recs;     // this job's state records
  uint32_t* hash;
  uint32_t* n_states;
  uint32_t cap;       // states this job may create (ids stay below ORIGIN_SELF - m)
  uint16_t* st;
  uint32_t row;
  bool accepting;
};


// Where the sets named by origin codes live, for the trie sweep of one job: a set index of the base
// chart (< m), m + k for local state k.  With ctx_below > 0 (the sweep of a root, whose chart's sets
// below its last one are placeholders) a completion that asks for such a set gets nothing and the
// step is flagged: its outcome depends on what the placeholder stands for.
constexpr uint32_t W_CTXHIT = 4;  // slot of WarpCtx::ctr
struct AutoView {
  const JobCtx& J;
  const AutoDev& A;
  uint32_t ctx_below;
  uint32_t* flag;  // shared-memory word (slot W_CTXHIT of the warp's counters)
  __device__ __forceinline__ void operator()(uint32_t o, const uint32_t*& p, uint32_t& n) const {
    if (o < ctx_below) {
      *flag = 1u;  // (every lane writes the same value)
      p = J.base_items;
      n = 0;
    } else if (o < J.m) {
      uint32_t a = J.base_off[o], b = J.base_off[o + 1];
      p = J.base_items + a;
      n = b - a;
    } else {
      const uint32_t* rec = J.recs + (size_t)(o - J.m) * A.rec_words;
      p = A.items + __ldcg(rec + AR_ITEMS);
      n = __ldcg(rec + AR_N);
    }
  }
  // an item of local state o that names its own state as origin means "origin o"
  __device__ __forceinline__ uint32_t fix(uint32_t item, uint32_t o) const {
    return ((item >> 16) == ORIGIN_SELF) ? ((o << 16) | (item & 0xFFFFu)) : item;
  }
  __device__ __forceinline__ void ctx_reset(const WarpCtx&) const {
    __syncwarp();
    if (ctx_below && lane_id() == 0) *flag = 0u;
    __syncwarp();
  }
  __device__ __forceinline__ bool ctx_hit(const WarpCtx&) const {
    __syncwarp();
    return ctx_below != 0u && *flag != 0u;
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
  WarpCtx w;
  uint32_t* tmp8;     // shared
  uint32_t n_computed = 0, n_created = 0;  // statistics, flushed once at the end of the kernel
  unsigned long long cycles = 0;           // SM cycles inside step()
  uint32_t chunk_at = 0, chunk_left = 0;   // this warp's private piece of the item pool (lane 0's copy counts)
  uint32_t gen = 1;                        // this fill's generation of the per-job hashes
  // Sets whose items name sets outside the chart (origin codes from region_base on: a frame's sets, or sets
  // of the walk's own, which may name a frame's sets in turn) mean different things in different frames:
  // such a set carries the frame as its "salt" and equals only sets with the same salt.  A set whose
  // origins all lie in the chart is the same set wherever it is met.
  uint32_t salt = 0, region_base = 0xffffffffu, eff_salt = 0;

  // A new set of job J with the items w.cur[0..n), the first nk of them its kernel: its id or T_FAIL.
  __device__ uint32_t create_set(const JobCtx& J, uint32_t n, uint32_t nk, uint32_t hash) {
    const uint32_t lane = lane_id();
    const AutoDev& A = S.au;
    uint32_t id = T_FAIL, ioff = 0;
    if (lane == 0) {
      const uint32_t got = atomicAdd(J.n_states, 1u);
      const uint32_t need = (max(n, 1u) + 31u) & ~31u;
      if (got < J.cap) {
        if (need > chunk_left) {  // take a new piece of the pool: one atomic per ~4 Ki item words
          const uint32_t take = max(need, 4096u);
          chunk_at = atomicAdd(&S.counters[CNT_AUTO_ITEMS], take);
          chunk_left = (chunk_at <= A.items_cap && take <= A.items_cap - chunk_at) ? take : 0u;
        }
        if (need <= chunk_left) {
          ioff = chunk_at;
          chunk_at += need;
          chunk_left -= need;
          id = got;
        } else {
          diag(S, DIAG_ITEM_POOL);
        }
      } else {
        diag(S, DIAG_SET_TABLE);
      }
    }
    id = __shfl_sync(FULL, id, 0);
    ioff = __shfl_sync(FULL, ioff, 0);
    if (id == T_FAIL) return T_FAIL;
    uint32_t* rec = J.recs + (size_t)id * A.rec_words;
    uint32_t* items = A.items + ioff;
    for (uint32_t i = lane; i < n; i += 32) items[i] = w.cur[i];
    for (uint32_t i = lane; i < A.rec_words; i += 32) {
      uint32_t v2 = 0u;
      if (i == AR_ITEMS) v2 = ioff;
      else if (i == AR_N) v2 = n;
      else if (i == AR_HASH) v2 = hash;
      else if (i == AR_NK) v2 = nk;
      else if (i == AR_SALT) v2 = eff_salt;
      else if (i >= AR_SCAN && i < AR_SCAN + 8) v2 = tmp8[i - AR_SCAN];
      else if (i >= AR_TRANS) v2 = T_UNKNOWN;
      rec[i] = v2;
    }
    __syncwarp();
    __threadfence();
    ++n_created;
    return id;
  }

  // Is set `sid` the one with this hash and a kernel of nk items for which `member` holds?
  // member(x, valid) is called by all lanes.
  template <class Member>
  __device__ __forceinline__ bool same_set(const JobCtx& J, uint32_t sid, uint32_t nk, uint32_t hash, Member member) {
    const uint32_t lane = lane_id();
    const uint32_t* rec = J.recs + (size_t)sid * S.au.rec_words;
    if (__ldcg(rec + AR_HASH) != hash || __ldcg(rec + AR_NK) != nk || __ldcg(rec + AR_SALT) != eff_salt) return false;
    const uint32_t* items = S.au.items + __ldcg(rec + AR_ITEMS);
    bool ok = true;
    for (uint32_t base = 0; base < nk; base += 32) {
      const bool valid = base + lane < nk;
      const uint32_t x = valid ? __ldcg(items + base + lane) : 0u;
      ok = member(x, valid) && ok;
    }
    return __all_sync(FULL, ok);
  }

  // The set of job J with this kernel: its id, or T_FAIL if there is none yet.
  // (A hash slot holds generation << 16 | id + 1; a slot of another generation, left by an earlier
  // fill, counts as empty, so the tables are never cleared between fills.)
  template <class Member>
  __device__ uint32_t lookup_set(const JobCtx& J, uint32_t nk, uint32_t hash, Member member) {
    const uint32_t lane = lane_id();
    const uint32_t mask = S.au.hash_mask;
    uint32_t slot = hash & mask;
    for (uint32_t probe = 0; probe <= mask && probe < 4096u; ++probe) {
      uint32_t v = 0;
      if (lane == 0) v = ld_acquire(&J.hash[slot]);
      v = __shfl_sync(FULL, v, 0);
      if ((v >> 16) != gen) break;
      if (same_set(J, (v & 0xFFFFu) - 1u, nk, hash, member)) return (v & 0xFFFFu) - 1u;
      slot = (slot + 1u) & mask;
    }
    return T_FAIL;
  }

  // Enter the freshly created set `id` into the job's hash, unless an equal set got there first
  // (several warps often reach the same new set at the same moment): returns the id to use.
  template <class Member>
  __device__ uint32_t insert_set(const JobCtx& J, uint32_t id, uint32_t nk, uint32_t hash, Member member) {
    const uint32_t lane = lane_id();
    const uint32_t mask = S.au.hash_mask;
    uint32_t slot = hash & mask;
    for (uint32_t probe = 0; probe <= mask && probe < 4096u; ++probe) {
      uint32_t old = 0;
      if (lane == 0) {
        old = ld_acquire(&J.hash[slot]);
        if ((old >> 16) != gen) {  // empty: take it, unless somebody is faster
          const uint32_t seen = old;
          old = atomicCAS(&J.hash[slot], seen, (gen << 16) | (id + 1u));
          if (old == seen) old = 0u;
        }
      }
      old = __shfl_sync(FULL, old, 0);
      if (old == 0u) return id;
      __threadfence();
      if (same_set(J, (old & 0xFFFFu) - 1u, nk, hash, member)) return (old & 0xFFFFu) - 1u;
      slot = (slot + 1u) & mask;
    }
    return T_FAIL;
  }

  // The kernel w.cur[0..nk) is new: predict, describe, store and enter the set.
  template <class Member>
  __device__ uint32_t finish_new(const JobCtx& J, uint32_t nk, uint32_t hash, Member member) {
    const uint32_t lane = lane_id();
    __syncwarp();
    if (lane == 0) w.ctr[W_NCUR] = nk, w.ctr[W_OVERFLOW] = 0u;
    predict_into_cur(G, w, ORIGIN_SELF);
    if (w.ctr[W_OVERFLOW]) return T_RETRY;
    const uint32_t n = min(w.ctr[W_NCUR], w.cur_cap);
    scannable_bytes(G, w.cur, n, tmp8);
    const uint32_t id = create_set(J, n, nk, hash);
    return id == T_FAIL ? T_FAIL : insert_set(J, id, nk, hash, member);
  }

  // The lane-resident form (see small_scan_complete) of the step from the set `pitems[0..plen)`,
  // whose own origin code is `pcode`, on `byte`.
  template <class View>
  __device__ uint32_t compute_small(const JobCtx& J, const View& view, const uint32_t* pitems, uint32_t plen, uint32_t pcode,
                                    uint32_t byte) {
    const uint32_t lane = lane_id();
    if (plen > 8u * 32u) return T_RETRY;  // a large set seldom scans into a small one
    uint32_t mine;
    bool accept;
    const uint32_t n = small_scan_complete(G, w, view, pitems, plen, byte, ORIGIN_SELF,
                                           [&](uint32_t it) { return view.fix(it, pcode); }, mine, accept);
    if (n == SMALL_OVERFLOW) return T_RETRY;
    if (n == 0) return T_DEAD;
    if (view.ctx_hit(w)) {  // a completion needed a set the walk does not know: the answer depends on the context
      clear_nt(G, w);
      return T_CTX;
    }
    // ---- the kernel: what is left when the completed items go
    const uint32_t nk = small_drop_completed(G, w, n, mine);
    uint32_t h = lane < nk ? mix32(mine) : 0u;
    for (int d = 16; d > 0; d >>= 1) h += __shfl_xor_sync(FULL, h, d);
    eff_salt = __any_sync(FULL, lane < nk && (mine >> 16) >= region_base && (mine >> 16) != ORIGIN_SELF) ? salt : 0u;
    h = mix32(h + nk * 0x9E3779B9u + eff_salt * 0x85EBCA77u);
    auto member = [&](uint32_t x, bool valid) {  // the kernel sits one item per lane
      bool found = false;
      for (uint32_t i = 0; i < nk; ++i)
        if (__shfl_sync(FULL, mine, i) == x) found = true;
      return found || !valid;
    };
    const uint32_t id = lookup_set(J, nk, h, member);
    if (id != T_FAIL) {
      clear_nt(G, w);
      return id;
    }
    return finish_new(J, nk, h, member);
  }

  // The general form, for sets of any size (w.cur may be the warp's large area).
  template <class View>
  __device__ uint32_t compute_general(const JobCtx& J, const View& view, const uint32_t* pitems, uint32_t plen,
                                      uint32_t pcode, uint32_t byte) {
    const uint32_t lane = lane_id();
    __syncwarp();
    if (lane < W_CTRS) w.ctr[lane] = 0u;
    __syncwarp();
    for (uint32_t k = lane; k < plen; k += 32) {
      const uint32_t it = pitems[k];
      const uint32_t inf = G.info[it & 0xFFFFu];
      const Scanned sc = scan_item(G, view.fix(it, pcode), inf, byte);
      if (sc.has_a) add_item(G, w, sc.a);
      if (sc.has_b) add_item(G, w, sc.b);
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
    if (view.ctx_hit(w)) {
      hset_clear_items(w, hashed);
      clear_nt(G, w);
      return T_CTX;
    }
    // the kernel: the items that are not completed; all of cur[0..hashed) are in the uniqueness hash
    uint32_t nk = 0, h = 0;
    bool reg = false;
    for (uint32_t base = 0; base < hashed; base += 32) {
      const uint32_t i = base + lane;
      const uint32_t it = i < hashed ? w.cur[i] : 0u;
      const bool keep = i < hashed && (G.info[it & 0xFFFFu] >> INFO_KIND_SHIFT) != KIND_END;
      if (keep) h += mix32(it);
      if (keep && (it >> 16) >= region_base && (it >> 16) != ORIGIN_SELF) reg = true;
      nk += __popc(__ballot_sync(FULL, keep));
    }
    for (int d = 16; d > 0; d >>= 1) h += __shfl_xor_sync(FULL, h, d);
    eff_salt = __any_sync(FULL, reg) ? salt : 0u;
    h = mix32(h + nk * 0x9E3779B9u + eff_salt * 0x85EBCA77u);
    auto member = [&](uint32_t x, bool valid) { return !valid || hset_contains(w.hset, w.hset_mask, x); };
    const uint32_t id = lookup_set(J, nk, h, member);
    if (id != T_FAIL) {
      hset_clear_items(w, hashed);
      clear_nt(G, w);
      return id;
    }
    // a new set: its items stay in the uniqueness hash, for the comparisons that entering the set
    // may need (the completed items among them do no harm: no stored kernel holds one)
    drop_completed(G, w, hashed);
    const uint32_t r = finish_new(J, nk, h, member);
    hset_clear_all(w.hset, w.hset_mask);
    return r == T_RETRY ? T_FAIL : r;
  }

  // One Earley step from the set `pitems[0..plen)` (own origin code `pcode`) on `byte`: T_DEAD, the id of
  // the set reached (in J's tables), T_CTX (only from a view that can say so), or T_FAIL when a capacity
  // was exceeded (the caller may switch to the large scratch and ask again).
  template <class View>
  __device__ uint32_t step(const JobCtx& J, const View& view, const uint32_t* pitems, uint32_t plen, uint32_t pcode,
                           uint32_t byte, bool small_ok) {
    const long long t0 = S.time_steps ? clock64() : 0;
    view.ctx_reset(w);
    uint32_t r = small_ok ? compute_small(J, view, pitems, plen, pcode, byte) : T_RETRY;
    if (r == T_RETRY) {
      view.ctx_reset(w);
      r = compute_general(J, view, pitems, plen, pcode, byte);
    }
    if (r != T_FAIL) ++n_computed;
    if (S.time_steps) cycles += (unsigned long long)(clock64() - t0);
    return r;
  }

  // The trie sweep's step: compute, publish and return the transition of local state `ps` on `byte`.
  // The transition has been claimed (T_PENDING) by whoever queued it.
  __device__ uint32_t compute(const JobCtx& J, uint32_t ps, uint32_t byte, bool small_ok) {
    const uint32_t* pitems;
    uint32_t plen;
    AutoView view{J, S.au, S.ctx_mode ? J.m - 1u : 0u, w.ctr + W_CTXHIT};
    const uint32_t pcode = ps == 0 ? J.m - 1 : J.m + ps;
    view(pcode, pitems, plen);
    const uint32_t r = step(J, view, pitems, plen, pcode, byte, small_ok);
    if (r == T_FAIL) return T_FAIL;
    uint32_t* slot = J.recs + (size_t)ps * S.au.rec_words + AR_TRANS + G.eq_of_byte[byte];
    if (lane_id() == 0) asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(slot), "r"(r) : "memory");
    return r;
  }
};

// How often a bounded wait polls before it gives up: 2^dflt times, or 2^poll_limit_shift when the state
// was created with a limit of its own (tests use a tiny one to take the give-up path).
__device__ __forceinline__ uint32_t poll_limit(const StateDev& S, uint32_t dflt) {
  return 1u << (S.poll_limit_shift ? S.poll_limit_shift : dflt);
}

// All CTAs of the (cooperatively launched) grid meet here.  Returns false if the sweep must be
// abandoned: some CTA waited longer than the limit, which only a fault elsewhere can cause.
__device__ __forceinline__ bool grid_barrier(const StateDev& S, uint32_t& phase) {
  __shared__ uint32_t ok_s;
  __syncthreads();
  if (threadIdx.x == 0) {
    ++phase;
    __threadfence();
    atomicAdd(&S.counters[CNT_BAR], 1u);
    const uint32_t target = phase * gridDim.x;
    uint32_t ok = 1u;
    for (uint32_t polls = 0;; ++polls) {
      if (ld_acquire(&S.counters[CNT_BAR]) >= target) break;
      if (polls > poll_limit(S, 24) || ld_acquire(&S.counters[CNT_BAR_ERR])) {
        if (polls > poll_limit(S, 24)) diag(S, DIAG_WAIT_GRID);
        atomicExch(&S.counters[CNT_BAR_ERR], 1u);
        ok = 0u;
        break;
      }
      __nanosleep(40);
    }
    __threadfence();
    ok_s = ok;
  }
  __syncthreads();
  const bool ok = ok_s != 0u;
  __syncthreads();
  return ok;
}

// A CTA reports that its part of a depth's pass is done (its writes are visible to whoever then sees
// the count) and goes on without waiting.  Returns false if the sweep is being abandoned.
__device__ __forceinline__ bool pass_arrive(const StateDev& S, uint32_t& phase) {
  __shared__ uint32_t go_s;
  __syncthreads();
  ++phase;  // (every thread keeps the count: the warps compare it with the global one on their own)
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(&S.counters[CNT_PASS_DONE], 1u);
    go_s = ld_acquire(&S.counters[CNT_BAR_ERR]) == 0u ? 1u : 0u;
  }
  __syncthreads();
  return go_s != 0u;
}


}  // namespace fmt
