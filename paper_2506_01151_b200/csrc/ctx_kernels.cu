// The mask fill (Sections 4.1, 4.3 of the paper: tokens whose validity does not depend on the context
// are looked up, only the context-dependent ones are checked against the parser state).
//
//   root_kernel       per computed row: its chart's last set with anonymous origins (a "root") is
//                     looked up in, or added to, the directory of roots
//   sweep_kernel      (kernels.cu, root mode) the trie sweep of every new root, once for good
//   collect_kernel    keeps a finished root sweep: mask row, region of sets, transition table
//   job_setup_kernel  rows whose root has no context-dependent trie node take the root's mask row;
//                     the others get their frame 0 and go to
//   fill_kernel       the level sweep over the trie, per (row, node): table look-ups inside frames,
//                     Earley steps against the row's own chart (Section 3.2) where the context matters
#include <cuda_runtime.h>

#include <algorithm>

#include "../../include/fmt.h"
#include "kernels.h"
#include "sweep_warp.cuh"

namespace fmt {

__device__ __forceinline__ void st_release64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_release32(uint32_t* p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// ===================================================================================== roots
//
// The last set of a pruned chart is sorted, origins ascending, and its own index is the largest origin
// there is, so the scanned / completed items (the set's kernel) come first and the predicted ones last.
// The start chart's only kernel item is the augmented start item.

constexpr int ROOT_WARPS = 8;
constexpr uint32_t ROOT_ITEMS = 1024;  // items of a last set that can become a root (staged in shared memory)

// Look a root up by its anonymous kernel `ab[0..nk)` (P placeholders; n items with the predicted ones
// `pred[0..n-nk)`, whose origins are replaced by P); add it if it is new and `may_add` (the protocol of
// the state cache: equal roots made at the same moment meet in the same slot and the loser adopts the
// winner's).  Returns the root's id or ROOT_NONE; `created` tells whether this call entered it.
// Called by all lanes with uniform arguments.
__device__ uint32_t root_find_or_add(const RootDev& R, const uint32_t* ab, const uint32_t* pred, uint32_t n, uint32_t nk,
                                     uint32_t P, uint32_t h, bool may_add, bool& created, uint32_t& chart_off) {
  const uint32_t lane = lane_id();
  created = false;
  chart_off = 0;
  uint32_t slot = h & R.hash_mask;
  int32_t my_id = -1;
  uint32_t my_chart = 0;
  for (uint32_t probe = 0; probe < 256; ++probe) {
    uint32_t v = 0;
    if (lane == 0) v = ld_acquire(&R.hash[slot]);
    v = __shfl_sync(FULL, v, 0);
    if (v == 0) {
      if (!may_add) return ROOT_NONE;
      if (my_id < 0) {
        int32_t id = -1;
        uint32_t coff = 0;
        const uint32_t words = CH_HDR + P + 2 + n, need = (words + 31u) & ~31u;
        if (lane == 0 && ld_acquire(R.n_roots) < R.max_roots && ld_acquire(&R.tops[TOP_CHARTS]) + need <= R.charts_cap) {
          const uint32_t got = atomicAdd(R.n_roots, 1u);
          if (got < R.max_roots) {
            coff = atomicAdd(&R.tops[TOP_CHARTS], need);
            if (coff <= R.charts_cap && need <= R.charts_cap - coff) id = (int32_t)got;
          }
        }
        id = __shfl_sync(FULL, id, 0);
        coff = __shfl_sync(FULL, coff, 0);
        if (id < 0) return ROOT_NONE;  // the directory is full
        uint32_t* c = R.charts + coff;  // a chart of P empty sets and the root set
        for (uint32_t i = lane; i < CH_HDR + P + 2; i += 32) {
          uint32_t v2 = 0u;
          if (i == CH_SETS) v2 = P + 1;
          else if (i == CH_ITEMS) v2 = n;
          else if (i == CH_WORDS) v2 = words;
          else if (i == CH_HDR + P + 1) v2 = n;
          c[i] = v2;
        }
        for (uint32_t i = lane; i < n; i += 32) c[CH_HDR + P + 2 + i] = i < nk ? ab[i] : ((P << 16) | (pred[i - nk] & 0xFFFFu));
        uint32_t* info = R.info + (size_t)id * RI_WORDS;
        if (lane < RI_WORDS) {
          uint32_t v2 = 0u;
          if (lane == RI_STATUS) v2 = ROOT_NEW;
          else if (lane == RI_P) v2 = P;
          else if (lane == RI_NK) v2 = nk;
          else if (lane == RI_N) v2 = n;
          else if (lane == RI_HASH) v2 = h;
          else if (lane == RI_CHART) v2 = coff;
          info[lane] = v2;
        }
        __syncwarp();
        __threadfence();
        my_id = id;
        my_chart = coff;
      }
      uint32_t old = 0;
      if (lane == 0) old = atomicCAS(&R.hash[slot], 0u, (uint32_t)my_id + 1u);
      old = __shfl_sync(FULL, old, 0);
      if (old == 0) {
        created = true;
        chart_off = my_chart;
        return (uint32_t)my_id;
      }
      v = old;
    }
    const uint32_t rid = v - 1u;
    if (rid >= R.max_roots) return ROOT_NONE;
    const uint32_t* info = R.info + (size_t)rid * RI_WORDS;
    bool same = __ldcg(info + RI_HASH) == h && __ldcg(info + RI_NK) == nk && __ldcg(info + RI_N) == n && __ldcg(info + RI_P) == P;
    if (same) {
      const uint32_t* c = R.charts + __ldcg(info + RI_CHART) + CH_HDR + P + 2;
      for (uint32_t i = lane; i < nk; i += 32)
        if (__ldcg(c + i) != ab[i]) same = false;
    }
    if (__all_sync(FULL, same)) {
      chart_off = __ldcg(info + RI_CHART);
      return rid;
    }
    slot = (slot + 1u) & R.hash_mask;
  }
  return ROOT_NONE;
}

// the root joins the roots this fill sweeps (one lane)
__device__ __forceinline__ void queue_root_sweep(const RootDev& R, uint32_t rid, uint32_t chart_off) {
  const uint32_t rj = atomicAdd(&R.counters[CNT_N_JOBS], 1u);
  R.rj_chart[rj] = chart_off;
  R.rj_mask[rj] = (int32_t)rid;
  R.rj_flags[rj] = 0u;
  R.rj_jobs[rj] = rj;
}

// Roots that a walk of the previous fills entered (it met a set that had no entry yet) are swept now, as
// far as this fill's own new roots leave room.
__global__ void pending_kernel(StateDev S) {
  const RootDev& R = S.rt;
  if (threadIdx.x != 0 || blockIdx.x != 0 || !R.on) return;
  const uint32_t np = min(R.tops[TOP_PENDING], R.pend_cap);
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  const uint32_t room = S.B > n_jobs ? S.B - n_jobs : 0u;
  const uint32_t take = min(np, room);
  for (uint32_t i = 0; i < take; ++i) {
    const uint32_t rid = R.pending[np - 1u - i];
    queue_root_sweep(R, rid, R.info[(size_t)rid * RI_WORDS + RI_CHART]);
  }
  R.tops[TOP_PENDING] = np - take;
}

// One warp per job: the row's root.
__global__ void __launch_bounds__(ROOT_WARPS * 32) root_kernel(GrammarDev G, StateDev S) {
  __shared__ uint32_t stage_all[ROOT_WARPS][ROOT_ITEMS];
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  const uint32_t warp = threadIdx.x >> 5, lane = lane_id();
  uint32_t* stage = stage_all[warp];
  const RootDev& R = S.rt;
  for (uint32_t j = blockIdx.x * ROOT_WARPS + warp; j < n_jobs; j += gridDim.x * ROOT_WARPS) {
    const uint32_t row = S.jobs[j];
    const uint64_t off = S.row_chart[row];
    const uint32_t* chart = S.arena + off;
    const uint32_t m = chart[CH_SETS];
    const uint32_t* items = chart + CH_HDR + m + 1;
    const uint32_t a = chart[CH_HDR + m - 1], b = chart[CH_HDR + m];
    const uint32_t n = b - a;
    uint32_t root = ROOT_NONE, P = 0, nk = 0;
    if (R.on && n > 0 && n <= min(R.max_items, ROOT_ITEMS)) {
      uint32_t h = 0;
      for (uint32_t base = 0; base < n; base += 32) {
        const uint32_t i = base + lane;
        const uint32_t it = i < n ? items[a + i] : 0u;
        const uint32_t o = it >> 16, r = it & 0xFFFFu;
        const bool is_k = i < n && (o != m - 1 || r == ITEM_START);
        const uint32_t prev_o = (i > 0 && i < n) ? (items[a + i - 1] >> 16) : 0xFFFFFFFFu;
        const bool newo = is_k && prev_o != o;
        const uint32_t nb = __ballot_sync(FULL, newo);
        const uint32_t rank = P + __popc(nb & ((1u << lane) - 1u)) - (newo ? 0u : 1u);  // the placeholder of this item's origin
        P += __popc(nb);
        nk += __popc(__ballot_sync(FULL, is_k));
        const uint32_t ab = ((is_k ? rank : P) << 16) | r;
        if (i < n) stage[i] = ab;
        if (is_k) h += mix32(ab);
        if (newo && rank < R.max_ph) S.cx.bind[(size_t)j * R.max_ph + rank] = (uint16_t)o;
      }
      for (int d = 16; d > 0; d >>= 1) h += __shfl_xor_sync(FULL, h, d);
      h = mix32(h + nk * 0x9E3779B9u) | 1u;
      __syncwarp();
      if (P >= 1 && P <= R.max_ph && nk >= 1) {
        bool created;
        uint32_t coff;
        root = root_find_or_add(R, stage, stage + nk, n, nk, P, h, true, created, coff);
        if (created && lane == 0) queue_root_sweep(R, root, coff);  // this fill sweeps it
      }
    }
    __syncwarp();
    if (lane == 0) {
      CtxJob cj;
      cj.chart_off = off;
      cj.m = m;
      cj.row_acc = row | ((chart[CH_FLAGS] & CHART_ACCEPTING) ? 0x80000000u : 0u);
      cj.root = root;
      cj.P = P;
      cj.spare[0] = cj.spare[1] = cj.spare[2] = 0;
      cj.mrow = S.row_mask[row];
      cj.pad[0] = cj.pad[1] = 0;
      S.cx.jobs[j] = cj;
    }
  }
}

// ===================================================================================== collect
//
// After the root sweep: one CTA per swept root keeps what later fills need.  The sweep left, per trie
// node, the set the node leads to (or dead / context-dependent) and, per set, its items and
// transitions.  Kept are the root's mask row (written by the sweep itself), the number of trie nodes
// marked context-dependent (none: the mask row is the whole answer for any row with this root), the
// items of every set (an Earley step of a row reads them with the row's bindings) and the
// transitions, as a table of 16-bit entries.

constexpr int COLLECT_THREADS = 1024;

// exclusive prefix sum over the block; returns this thread's offset, `total` gets the block's sum
__device__ __forceinline__ uint32_t block_scan(uint32_t v, uint32_t* warp_sums /* [33] shared */, uint32_t& total) {
  const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
  uint32_t incl = v;
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t t = __shfl_up_sync(FULL, incl, d);
    if ((int)lane >= d) incl += t;
  }
  __syncthreads();
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t w = lane < (blockDim.x >> 5) ? warp_sums[lane] : 0u;
    uint32_t wi = w;
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t t = __shfl_up_sync(FULL, wi, d);
      if ((int)lane >= d) wi += t;
    }
    warp_sums[lane] = wi - w;
    if (lane == 31) warp_sums[32] = wi;
  }
  __syncthreads();
  total = warp_sums[32];
  return warp_sums[warp] + incl - v;
}

__global__ void __launch_bounds__(COLLECT_THREADS) collect_kernel(GrammarDev G, StateDev S) {
  const RootDev& R = S.rt;
  const AutoDev& A = S.au;
  const uint32_t rj = blockIdx.x;
  if (rj >= R.counters[CNT_N_JOBS]) return;
  __shared__ uint32_t sums[33];
  __shared__ uint32_t sh[5];
  __shared__ uint8_t rep_byte[256];
  const uint32_t rid = (uint32_t)R.rj_mask[rj];
  uint32_t* info = R.info + (size_t)rid * RI_WORDS;
  const uint32_t P = info[RI_P], n_root = info[RI_N];
  const uint32_t* chart = R.charts + info[RI_CHART];
  const uint16_t* st = A.st + (size_t)rj * A.st_stride;
  const uint32_t* recs = A.recs + (size_t)rj * A.cap * A.rec_words;
  // (the ids the sweep could hand out: as in its own job set-up)
  const uint32_t id_cap = min(min(A.cap, ORIGIN_SELF - 2u - P), ORIGIN_SELF - 16u - RBASE);
  const uint32_t nst = min(A.n_states[rj], id_cap);
  bool failed = R.counters[CNT_BAR_ERR] != 0u || (R.rj_flags[rj] & ROW_BROKEN) != 0u || nst == 0u;
  const uint32_t visited_end = G.lvl_off[min(R.counters[CNT_LAST_LEVEL], G.depth) + 1];
  auto frontier_at = [&](uint32_t node, uint32_t& ps) -> bool {
    const uint32_t s = st[node];
    if (s != ST_CTX && s != ST_PENDING) return false;
    const uint32_t p = G.parent[node];
    ps = (p == 0) ? 0u : (uint32_t)st[p];
    return true;
  };
  // ---- pass 1: how many frontier nodes, how many items
  uint32_t cnt = 0, bad = 0;
  for (uint32_t node = 1 + threadIdx.x; node < visited_end; node += blockDim.x) {
    uint32_t ps;
    if (frontier_at(node, ps)) {
      ++cnt;
      if (ps >= nst) bad = 1;  // (a node left waiting below a parent that is not a set: cannot happen; do not trust the sweep then)
    }
  }
  uint32_t n_items = 0;
  for (uint32_t k = threadIdx.x; k < nst; k += blockDim.x) n_items += (k == 0) ? n_root : recs[(size_t)k * A.rec_words + AR_N];
  uint32_t fr_total, it_total, bad_total;
  block_scan(cnt, sums, fr_total);
  block_scan(n_items, sums, it_total);
  block_scan(bad, sums, bad_total);
  if (bad_total) failed = true;
  const uint32_t tr_total = nst * G.n_eq;
  if (threadIdx.x == 0) {
    uint32_t fo = 0, so = 0, io = 0, to = 0, f = failed ? 1u : 0u;
    if (!f) {
      so = atomicAdd(&R.tops[TOP_STATES], nst);
      io = atomicAdd(&R.tops[TOP_ITEMS], it_total);
      to = atomicAdd(&R.tops[TOP_TRANS], tr_total);
      if (so > R.st_cap || nst > R.st_cap - so || io > R.it_cap || it_total > R.it_cap - io ||
          to > R.tr_cap || tr_total > R.tr_cap - to)
        f = 1u;
    }
    sh[0] = fo, sh[1] = so, sh[2] = io, sh[3] = f, sh[4] = to;
  }
  if (threadIdx.x < 256) rep_byte[threadIdx.x] = 0u;
  __syncthreads();
  if (threadIdx.x < 256) rep_byte[G.eq_of_byte[threadIdx.x]] = (uint8_t)threadIdx.x;  // any byte of the class will do
  __syncthreads();
  const uint32_t st_off = sh[1], it_off = sh[2], tr_off = sh[4];
  failed = sh[3] != 0u;
  if (!failed) {
    // ---- the region: where each set's items go, then the items
    uint32_t run = 0;
    for (uint32_t base = 0; base < nst; base += blockDim.x) {
      const uint32_t k = base + threadIdx.x;
      const uint32_t nk = k < nst ? ((k == 0) ? n_root : recs[(size_t)k * A.rec_words + AR_N]) : 0u;
      uint32_t tile;
      const uint32_t at = block_scan(nk, sums, tile);
      if (k < nst) R.states[st_off + k] = make_uint2(it_off + run + at, nk);
      run += tile;
    }
    __syncthreads();
    const uint32_t warp = threadIdx.x >> 5, lane = lane_id();
    for (uint32_t k = warp; k < nst; k += blockDim.x >> 5) {
      const uint2 e = R.states[st_off + k];
      const uint32_t* src = (k == 0) ? chart + CH_HDR + P + 2 : A.items + recs[(size_t)k * A.rec_words + AR_ITEMS];
      for (uint32_t i = lane; i < e.y; i += 32) R.items[e.x + i] = src[i];
    }
    // ---- the region's transitions, one 16-bit entry per (set, byte class).  A transition the sweep never
    // asked for is dead when the set cannot scan the byte, else left to the rows' own walks.
    for (uint32_t i = threadIdx.x; i < tr_total; i += blockDim.x) {
      const uint32_t k = i / G.n_eq, e = i % G.n_eq;
      const uint32_t* rec = recs + (size_t)k * A.rec_words;
      const uint32_t t = rec[AR_TRANS + e], b = rep_byte[e];
      uint16_t v;
      if (t == T_DEAD) v = R_DEAD;
      else if (t < nst) v = (uint16_t)t;
      else if (t == T_UNKNOWN && !((rec[AR_SCAN + (b >> 5)] >> (b & 31u)) & 1u)) v = R_DEAD;
      else v = R_CTX;
      R.trans[tr_off + i] = v;
    }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    info[RI_FR_N] = failed ? 0u : fr_total;
    info[RI_ST_OFF] = st_off;
    info[RI_TR_OFF] = tr_off;
    info[RI_NSTATES] = failed ? 0u : nst;
    __threadfence();
    info[RI_STATUS] = failed ? ROOT_FAILED : ROOT_READY;
    if (failed) diag(S, DIAG_ROOT_FAILED);
    stat_add(S, CNT_STAT_ROOT_SWEEPS, 1u);
  }
}

// ===================================================================================== fill: set-up
//
// One CTA per job.  A job whose root has been swept and has no context-dependent trie node at all
// takes the root's mask row as it is (plus the EOS bit of an accepting chart): Section 4.3's
// context-independent mask, and nothing else to do.  Every other job goes to the level sweep: with
// frame 0 (its root's region, placeholders bound as root_kernel found them) if it has a root, from
// the chart's own last set if not.

__global__ void __launch_bounds__(256) job_setup_kernel(GrammarDev G, StateDev S) {
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  const RootDev& R = S.rt;
  const uint32_t Wm = G.Wm;
  for (uint32_t j = blockIdx.x; j < n_jobs; j += gridDim.x) {
    const CtxJob cj = S.cx.jobs[j];
    const uint32_t* info = R.info + (size_t)(cj.root != ROOT_NONE ? cj.root : 0u) * RI_WORDS;
    const bool use = cj.root != ROOT_NONE && __ldcg(info + RI_STATUS) == ROOT_READY;
    if (use && __ldcg(info + RI_FR_N) == 0u) {
      const uint32_t* src = R.ci_rows + (size_t)cj.root * Wm;
      uint32_t* dst = S.mask_rows + (size_t)cj.mrow * Wm;
      const bool acc = (cj.row_acc >> 31) != 0u && G.eos >= 0;
      for (uint32_t w = threadIdx.x; w < Wm; w += blockDim.x) {
        uint32_t v = src[w];
        if (acc && w == ((uint32_t)G.eos >> 5)) v |= 1u << ((uint32_t)G.eos & 31u);
        dst[w] = v;
      }
      if (threadIdx.x == 0) stat_add(S, CNT_STAT_JOBS_MASK, 1u);
      continue;
    }
    if (threadIdx.x == 0) {
      Frame f;
      f.root = cj.root, f.P = cj.P, f.n = use ? info[RI_NSTATES] : 0u;
      f.st_off = use ? info[RI_ST_OFF] : 0u, f.tr_off = use ? info[RI_TR_OFF] : 0u, f.pad0 = f.pad1 = f.pad2 = 0u;
      S.cx.frames[(size_t)j * MAXF] = f;
      S.cx.frame_ctr[j] = use ? 1u : 0u;
      S.cx.jobs[j].pad[0] = use ? 1u : 0u;
      S.au.n_states[j] = 0u;
      S.cx.fjobs[atomicAdd(&S.counters[CNT_N_FJOBS], 1u)] = j;
      stat_add(S, use ? CNT_STAT_JOBS_ROOT : CNT_STAT_JOBS_PLAIN, 1u);
    }
    if (use)
      for (uint32_t i = threadIdx.x; i < cj.P && i < R.max_ph; i += blockDim.x)
        S.cx.fbind[(size_t)j * MAXF * R.max_ph + i] = S.cx.bind[(size_t)j * R.max_ph + i];
  }
}

// ===================================================================================== walk
//
// Origin codes of the sets a job's walk meets (see RootDev): a set of the row's chart, a set made by
// this walk, or a set of a frame.  Items read from a frame's set carry the root's anonymous origins:
// placeholders are replaced by the chart sets the frame binds them to.
struct WalkView {
  const uint32_t* base_off;
  const uint32_t* base_items;
  const uint32_t* lrecs;  // the sets this walk has made
  uint32_t rec_words;
  const uint32_t* litems;
  const Frame* cur;          // the frame that the codes from RBASE on mean in this step (or nullptr)
  const uint16_t* cur_bind;  // what its placeholders stand for
  const uint2* rstates;      // the roots' pools
  const uint32_t* ritems;
  __device__ __forceinline__ void operator()(uint32_t o, const uint32_t*& p, uint32_t& n) const {
    if (o < LBASE) {
      const uint32_t a = base_off[o], b = base_off[o + 1];
      p = base_items + a;
      n = b - a;
    } else if (o < RBASE) {
      const uint32_t* rec = lrecs + (size_t)(o - LBASE) * rec_words;
      p = litems + __ldcg(rec + AR_ITEMS);
      n = __ldcg(rec + AR_N);
    } else {
      const uint2 e = __ldg(rstates + __ldcg(&cur->st_off) + (o - RBASE));
      p = ritems + e.x;
      n = e.y;
    }
  }
  // an item read from set o, in the walk's own naming
  __device__ __forceinline__ uint32_t fix(uint32_t item, uint32_t o) const {
    if (o < LBASE) return item;
    uint32_t oo = item >> 16;
    if (o < RBASE) return (oo == ORIGIN_SELF) ? ((o << 16) | (item & 0xFFFFu)) : item;
    const uint32_t P = __ldcg(&cur->P);
    if (oo == ORIGIN_SELF) oo = o;
    else if (oo < P) oo = __ldcg(cur_bind + oo);
    else if (oo == P) oo = RBASE;               // the root set is set 0 of its region
    else oo = RBASE + (oo - P - 1u);            // the root sweep named its k-th set P + 1 + k
    return (oo << 16) | (item & 0xFFFFu);
  }
  __device__ __forceinline__ void ctx_reset(const WarpCtx&) const {}
  __device__ __forceinline__ bool ctx_hit(const WarpCtx&) const { return false; }
};

constexpr uint32_t NOF = 0xffffffffu;                       // "no frame"
constexpr uint32_t V_DEAD = 0xFFFFu, V_PEND = 0xFFFEu;      // values of a remembered transition (16 bits)
constexpr uint32_t CODE_CHART = 0xFFFFu;                    // "parent set" of a job without a root: the chart's last set

struct Walker {
  const GrammarDev& G;
  const StateDev& S;
  SweepWarp& sw;
  uint32_t* big;
  bool big_mode = false;
  uint32_t n_frames = 0;

  __device__ __forceinline__ JobCtx job(const CtxJob& cj, uint32_t j) const {
    const AutoDev& A = S.au;
    JobCtx J;
    const uint32_t* chart = S.arena + cj.chart_off;
    J.row = cj.row_acc & 0x7FFFFFFFu;
    J.accepting = (cj.row_acc >> 31) != 0u;
    J.m = cj.m;
    J.base_off = chart + CH_HDR;
    J.base_items = chart + CH_HDR + cj.m + 1;
    J.recs = A.recs + (size_t)j * A.cap * A.rec_words;
    J.hash = A.hash + (size_t)j * (A.hash_mask + 1);
    J.n_states = A.n_states + j;
    J.cap = min(A.cap, RBASE - LBASE);
    J.st = nullptr;
    return J;
  }
  __device__ __forceinline__ WalkView view(const JobCtx& J, uint32_t j, uint32_t frame) const {
    WalkView v;
    v.base_off = J.base_off;
    v.base_items = J.base_items;
    v.lrecs = J.recs;
    v.rec_words = S.au.rec_words;
    v.litems = S.au.items;
    v.cur = frame == NOF ? nullptr : S.cx.frames + (size_t)j * MAXF + frame;
    v.cur_bind = frame == NOF ? nullptr : S.cx.fbind + ((size_t)j * MAXF + frame) * S.rt.max_ph;
    v.rstates = S.rt.states;
    v.ritems = S.rt.items;
    return v;
  }
  __device__ void break_row(const JobCtx& J) {
    if (lane_id() == 0) {
      if (!(atomicOr(&S.row_flags[J.row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
      atomicExch(&S.counters[CNT_ERR], 1u);
    }
  }
  // One Earley step of job j from the set with origin code `pcode`, which lives in `frame` (or NOF),
  // on `byte` (all lanes, uniform arguments): the id of the set reached, or T_DEAD (also when a
  // capacity ran out: the row is marked broken then, its mask is not used).
  __device__ uint32_t step(const CtxJob& cj, uint32_t j, uint32_t pcode, uint32_t frame, uint32_t byte) {
    const JobCtx J = job(cj, j);
    const WalkView v = view(J, j, frame);
    sw.salt = frame == NOF ? 0u : frame + 1u;
    sw.region_base = LBASE;  // (a set that names sets of the walk's own may depend on the frame through them)
    const uint32_t* pitems;
    uint32_t plen;
    v(pcode, pitems, plen);
    uint32_t r = sw.step(J, v, pitems, plen, pcode, byte, !big_mode);
    if (r == T_FAIL && !big_mode) {  // a set outgrew the shared-memory scratch: use the large area from now on
      big_mode = true;
      hset_clear_all(sw.w.hset, sw.w.hset_mask);
      clear_nt(G, sw.w);
      sw.w.cur = big;
      sw.w.cur_cap = S.big_arena_items;
      sw.w.hset = big + S.big_arena_items;
      sw.w.hset_mask = S.big_hset_slots - 1;
      if (lane_id() == 0) stat_add(S, CNT_STAT_BIG, 1u);
      r = sw.step(J, v, pitems, plen, pcode, byte, false);
    }
    if (r == T_FAIL) {
      hset_clear_all(sw.w.hset, sw.w.hset_mask);
      clear_nt(G, sw.w);
      if (lane_id() == 0) diag(S, DIAG_SET_SCRATCH);
      break_row(J);
      r = T_DEAD;
    }
    return r;
  }
};

// Is the set `id` this walk made itself a known root, with all its origins in the row's chart?  Then
// what follows it is context-independent again: the job gets a frame for it (the root's region with
// the placeholders bound to those chart sets) and the set is walked by table look-ups from there on.
// Returns frame + 1 or NOFRAME, and remembers the answer in the set's record.  Called by all lanes
// with uniform arguments, between Earley steps (it uses the warp's set scratch).
__device__ uint32_t resolve_frame(Walker& wk, const CtxJob& cj, uint32_t j, uint32_t id) {
  const StateDev& S = wk.S;
  const RootDev& R = S.rt;
  const AutoDev& A = S.au;
  const uint32_t lane = lane_id();
  uint32_t* rec = A.recs + ((size_t)j * A.cap + id) * A.rec_words;
  const uint32_t nk = __ldcg(rec + AR_NK), n = __ldcg(rec + AR_N);
  const uint32_t* items = A.items + __ldcg(rec + AR_ITEMS);
  uint32_t result = NOFRAME;
  constexpr uint32_t KMAX = 256;  // (the scratch has 512 words: the sorted kernel, then its anonymous form)
  if (R.on && nk >= 1 && nk <= KMAX && n <= R.max_items && wk.sw.w.cur_cap >= 2 * KMAX) {
    uint32_t* buf = wk.sw.w.cur;
    uint32_t* abs_items = buf + KMAX;
    bool ok = true;
    __syncwarp();
    for (uint32_t i = lane; i < nk; i += 32) {
      const uint32_t it = __ldcg(items + i);
      buf[i] = it;
      if ((it >> 16) >= LBASE) ok = false;  // an origin inside the token: not a situation a chart can be in
    }
    ok = __all_sync(FULL, ok);
    if (ok) {
      sort_items(buf, nk, KMAX);
      __syncwarp();
      uint32_t P = 0, h = 0;
      for (uint32_t base = 0; base < nk; base += 32) {
        const uint32_t i = base + lane;
        const uint32_t it = i < nk ? buf[i] : 0u;
        const uint32_t o = it >> 16;
        const uint32_t prev_o = (i > 0 && i < nk) ? (buf[i - 1] >> 16) : 0xFFFFFFFFu;
        const bool newo = i < nk && prev_o != o;
        const uint32_t nb = __ballot_sync(FULL, newo);
        const uint32_t rank = P + __popc(nb & ((1u << lane) - 1u)) - (newo ? 0u : 1u);
        P += __popc(nb);
        if (i < nk) {
          const uint32_t ab = (rank << 16) | (it & 0xFFFFu);
          abs_items[i] = ab;
          h += mix32(ab);
        }
      }
      for (int d = 16; d > 0; d >>= 1) h += __shfl_xor_sync(FULL, h, d);
      h = mix32(h + nk * 0x9E3779B9u) | 1u;
      __syncwarp();
      if (P >= 1 && P <= R.max_ph) {
        bool created;
        uint32_t coff;
        // (a set without an entry gets one: the next fill sweeps it, this walk goes on by Earley steps)
        // (one lane looks, all lanes act on what it saw: the count moves while other warps add to the list)
        uint32_t room_ = 0;
        if (lane == 0) room_ = ld_acquire(&R.tops[TOP_PENDING]) < R.pend_cap ? 1u : 0u;
        const bool room = __shfl_sync(FULL, room_, 0) != 0u;
        const uint32_t rid = root_find_or_add(R, abs_items, items + nk, n, nk, P, h, room, created, coff);
        if (created && lane == 0) {
          const uint32_t at = atomicAdd(&R.tops[TOP_PENDING], 1u);
          if (at < R.pend_cap) R.pending[at] = rid;
        }
        if (rid != ROOT_NONE) {
          const uint32_t* info = R.info + (size_t)rid * RI_WORDS;
          const uint32_t nst = __ldcg(info + RI_NSTATES);
          if (ld_acquire(info + RI_STATUS) == ROOT_READY && nst > 0) {
            uint32_t idx = 0;
            if (lane == 0) idx = atomicAdd(S.cx.frame_ctr + j, 1u);
            idx = __shfl_sync(FULL, idx, 0);
            if (idx < MAXF) {
              Frame* f = S.cx.frames + (size_t)j * MAXF + idx;
              if (lane == 0) {
                Frame nf;
                nf.root = rid, nf.P = P, nf.n = nst;
                nf.st_off = __ldcg(info + RI_ST_OFF), nf.tr_off = __ldcg(info + RI_TR_OFF), nf.pad0 = nf.pad1 = nf.pad2 = 0u;
                *f = nf;
              }
              uint16_t* fb = S.cx.fbind + ((size_t)j * MAXF + idx) * R.max_ph;
              for (uint32_t i = lane; i < nk; i += 32) {  // the chart set each placeholder stands for
                const uint32_t r = abs_items[i] >> 16;
                if (i == 0 || (abs_items[i - 1] >> 16) != r) fb[r] = (uint16_t)(buf[i] >> 16);
              }
              __syncwarp();
              __threadfence();
              result = idx + 1u;
              ++wk.n_frames;
            }
          }
        }
      }
    }
  }
  uint32_t old = 0;
  if (lane == 0) old = atomicCAS(rec + AR_FRAME, 0u, result);
  old = __shfl_sync(FULL, old, 0);
  return old != 0u ? old : result;  // (another warp may have looked the same set up meanwhile: use its answer)
}

// ===================================================================================== fill: level sweep with frames
//
// The fill proper.  Like the root sweep it goes through the trie one depth at a time, one THREAD per
// (job, node): node's set = transition(parent's set, byte), with coalesced reads of the trie and
// writes of the per-node sets, the depths overlapped by tickets as in sweep_kernel.  The difference
// is where a transition comes from.  A job starts in set 0 of its frame 0 (its root's region); inside
// a frame a transition is ONE look-up in the root's table, shared by all rows and fills; only where
// the table says "context-dependent" is an Earley step run against the row's chart (queued, computed
// by a warp, remembered per job), and the set it yields usually opens the next frame.  Jobs without a
// root start from the chart's last set and do everything by Earley steps, as does whatever set has
// no frame.
//
// A node's word: SS_DEAD, SS_PENDING (its transition is queued), or (frame + 1) << 16 | code, with
// frame + 1 = 0 for a set of the walk's own (code = LBASE + id) and for the chart's last set (CODE_CHART).
constexpr uint32_t SS_DEAD = 0xffffffffu, SS_PENDING = 0xfffffffeu, SS_CLAIMED = 0xfffffffdu;

struct FillReq {
  uint32_t frame1, code;  // the parent set of the transition this thread has just claimed
};

// (one thread) The set job j reaches from `state` on `byte`; SS_PENDING if somebody is computing it;
// SS_CLAIMED if nobody had asked yet and `claim` is set: the caller must queue `rq`.
__device__ uint32_t fill_next(const GrammarDev& G, const StateDev& S, uint32_t j, uint32_t state, uint32_t byte, bool claim, FillReq& rq) {
  const AutoDev& A = S.au;
  const uint32_t eq = G.eq_of_byte[byte];
  uint32_t frame1 = state >> 16, code = state & 0xFFFFu;
  if (frame1 == 0u && code != CODE_CHART) {  // a set of the walk's own
    uint32_t* rec = A.recs + ((size_t)j * A.cap + (code - LBASE)) * A.rec_words;
    const uint32_t fr = __ldcg(rec + AR_FRAME);  // (looked up by whoever made the set, before its id went anywhere)
    if (fr != 0u && fr != NOFRAME) {
      frame1 = fr, code = RBASE;  // it opens a frame: go on in that frame's table
    } else {
      if (!((__ldcg(rec + AR_SCAN + (byte >> 5)) >> (byte & 31u)) & 1u)) return SS_DEAD;
      uint32_t* slot = rec + AR_TRANS + eq;
      uint32_t t = ld_acquire(slot);
      if (t == T_UNKNOWN && claim) {
        t = atomicCAS(slot, T_UNKNOWN, T_PENDING);
        if (t == T_UNKNOWN) {
          rq.frame1 = 0u, rq.code = code;
          return SS_CLAIMED;
        }
      }
      if (t == T_PENDING || t == T_UNKNOWN) return SS_PENDING;
      return t == T_DEAD ? SS_DEAD : LBASE + t;
    }
  }
  if (frame1 != 0u) {  // a frame's set: the root's table
    const Frame* f = S.cx.frames + (size_t)j * MAXF + (frame1 - 1u);
    const uint32_t t16 = __ldg(S.rt.trans + __ldcg(&f->tr_off) + (size_t)(code - RBASE) * G.n_eq + eq);
    if (t16 == R_DEAD) return SS_DEAD;
    if (t16 < R_CTX) return (frame1 << 16) | (RBASE + t16);
  }
  // ---- context-dependent (or out of the chart's last set): the job's own table
  const unsigned long long gen = S.gen_ctx & 0xFFFFu;
  const unsigned long long key = ((unsigned long long)(frame1 & 0xFFu) << 24) | (code << 8) | eq;
  unsigned long long* tab = S.cx.ctab + (size_t)j * CT_SLOTS;
  uint32_t s = mix32((uint32_t)key) & (CT_SLOTS - 1);
  for (uint32_t probe = 0; probe < 128; ++probe) {
    unsigned long long v = ld_acquire64(tab + s);
    if ((v >> 48) != gen) {  // left by an earlier fill: free
      if (!claim) return SS_PENDING;
      const unsigned long long old = atomicCAS(tab + s, v, (gen << 48) | (key << 16) | V_PEND);
      if (old == v) {
        rq.frame1 = frame1, rq.code = code;
        return SS_CLAIMED;
      }
      v = old;
      if ((v >> 48) != gen) {
        --probe;
        continue;
      }
    }
    if (((v >> 16) & 0xFFFFFFFFull) == key) {
      const uint32_t val = (uint32_t)v & 0xFFFFu;
      return val == V_PEND ? SS_PENDING : val == V_DEAD ? SS_DEAD : LBASE + val;
    }
    s = (s + 1u) & (CT_SLOTS - 1);
  }
  // no room to remember the transition: give the row up rather than guess
  const uint32_t row = S.cx.jobs[j].row_acc & 0x7FFFFFFFu;
  if (!(atomicOr(&S.row_flags[row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
  atomicExch(&S.counters[CNT_ERR], 1u);
  diag(S, DIAG_SET_TABLE);
  return SS_DEAD;
}

// (one lane) The transition (frame1, code, eq) of job j, which some thread claimed, is `val` (a set id or V_DEAD).
__device__ void fill_publish(const StateDev& S, uint32_t j, uint32_t frame1, uint32_t code, uint32_t eq, uint32_t val) {
  const AutoDev& A = S.au;
  if (frame1 == 0u && code != CODE_CHART) {
    uint32_t* slot = A.recs + ((size_t)j * A.cap + (code - LBASE)) * A.rec_words + AR_TRANS + eq;
    st_release32(slot, val == V_DEAD ? T_DEAD : val);
    return;
  }
  const unsigned long long gen = S.gen_ctx & 0xFFFFu;
  const unsigned long long key = ((unsigned long long)(frame1 & 0xFFu) << 24) | (code << 8) | eq;
  unsigned long long* tab = S.cx.ctab + (size_t)j * CT_SLOTS;
  uint32_t s = mix32((uint32_t)key) & (CT_SLOTS - 1);
  for (uint32_t probe = 0; probe < 128; ++probe) {
    const unsigned long long v = ld_acquire64(tab + s);
    if ((v >> 48) == gen && ((v >> 16) & 0xFFFFFFFFull) == key) {
      st_release64(tab + s, (gen << 48) | (key << 16) | val);
      return;
    }
    s = (s + 1u) & (CT_SLOTS - 1);
  }
}

constexpr uint32_t FILL_PER_LANE = 4;  // trie nodes per lane and pass iteration (independent loads in flight)

__global__ void __launch_bounds__(SWEEP_WARPS * 32, 1) fill_kernel(GrammarDev Gg, StateDev S) {
  const uint32_t n_jobs = S.counters[CNT_N_FJOBS];  // (the jobs that need the sweep: S.cx.fjobs)
  if (n_jobs == 0) return;  // every CTA sees the same count: nobody is left at a barrier
  extern __shared__ __align__(16) uint32_t smem[];
  const uint32_t warp = threadIdx.x >> 5, lane = lane_id();
  const AutoDev& A = S.au;
  const uint32_t ntw = (2u * Gg.Nw + 7u) & ~7u;
  const uint32_t warp_words = SWEEP_CUR + SWEEP_HSET + ntw + W_CTRS + 8;
  uint32_t* mine = smem + (size_t)warp * warp_words;
  GrammarDev G = Gg;
  if (A.tables_in_smem) G = stage_hot_tables(Gg, smem + (size_t)SWEEP_WARPS * warp_words);
  SweepWarp sw{G, S};
  sw.gen = S.gen_ctx & 0xFFFFu;
  sw.w.cur = mine;
  sw.w.cur_cap = SWEEP_CUR;
  sw.w.hset = mine + SWEEP_CUR;
  sw.w.hset_mask = SWEEP_HSET - 1;
  sw.w.nt = sw.w.hset + SWEEP_HSET;
  sw.w.ctr = sw.w.nt + ntw;
  sw.tmp8 = sw.w.ctr + W_CTRS;
  hset_clear_all(sw.w.hset, SWEEP_HSET - 1);
  for (uint32_t i = lane; i < ntw; i += 32) sw.w.nt[i] = 0u;
  if (lane < W_CTRS) sw.w.ctr[lane] = 0u;
  __syncthreads();
  Walker wk{G, S, sw, S.big_scratch + ((size_t)blockIdx.x * SWEEP_WARPS + warp) * ((size_t)S.big_arena_items + S.big_hset_slots)};
  const uint32_t gw = blockIdx.x * SWEEP_WARPS + warp, GW = gridDim.x * SWEEP_WARPS;
  uint32_t pass_phase = 0;
  const uint32_t stride = A.st_stride;
  const unsigned long long gen = S.gen_ctx & 0xFFFFu;

  uint32_t last_level = 0;
  uint32_t expect_req = n_jobs * Gg.n_eq;
  for (uint32_t L = 1; L <= G.depth; ++L) {
    const uint32_t lo = __ldg(&G.lvl_off[L]), hi = __ldg(&G.lvl_off[L + 1]);
    constexpr uint32_t CH = 32 * FILL_PER_LANE;
    const uint32_t nL = hi - lo, cpj = (nL + CH - 1) / CH;
    const uint32_t chunks = n_jobs * cpj;
    bool any_alive = false;
    const uint32_t req_half = S.cx.req2_cap / 2u, req_base = (L & 1u) * req_half;
    for (uint32_t c = gw; c < chunks; c += GW) {
      const uint32_t ji = c / cpj, j = __ldg(&S.cx.fjobs[ji]);
      const uint32_t first = lo + (c % cpj) * CH + lane;
      uint32_t* st = S.cx.st32 + (size_t)ji * stride;
      const uint32_t start = __ldcg(&S.cx.jobs[j].pad[0]) ? ((1u << 16) | RBASE) : CODE_CHART;  // set 0 of frame 0, or the chart's last set
      uint32_t node[FILL_PER_LANE], byte[FILL_PER_LANE], par[FILL_PER_LANE], ps[FILL_PER_LANE];
#pragma unroll
      for (uint32_t u = 0; u < FILL_PER_LANE; ++u) {
        node[u] = first + 32u * u;
        const bool v = node[u] < hi;
        byte[u] = v ? __ldg(&G.node_byte[node[u]]) : 0u;
        par[u] = (v && L > 1) ? __ldg(&G.parent[node[u]]) : 0u;
      }
#pragma unroll
      for (uint32_t u = 0; u < FILL_PER_LANE; ++u) ps[u] = (node[u] < hi) ? ((L == 1) ? start : __ldcg(st + par[u])) : SS_DEAD;
#pragma unroll
      for (uint32_t u = 0; u < FILL_PER_LANE; ++u) {
        if (node[u] >= hi) continue;
        uint32_t p_state = ps[u];
        FillReq rq;
        if (p_state == SS_PENDING) {  // settle the parent first: its transition was queued at the depth before
          const uint32_t gp_state = (L == 2) ? start : __ldcg(st + __ldg(&G.parent[par[u]]));
          const uint32_t pbyte = __ldg(&G.node_byte[par[u]]);
          uint32_t t2 = (gp_state == SS_DEAD || gp_state == SS_PENDING) ? SS_DEAD : fill_next(G, S, j, gp_state, pbyte, false, rq);
          for (uint32_t spin = 0; t2 == SS_PENDING && spin < poll_limit(S, 21); ++spin) {
            __nanosleep(40);
            t2 = fill_next(G, S, j, gp_state, pbyte, false, rq);
          }
          if (t2 == SS_PENDING) {  // the wait ran out: give the row up rather than guess
            diag(S, DIAG_WAIT_VALUE);
            const uint32_t row = __ldcg(&S.cx.jobs[j].row_acc) & 0x7FFFFFFFu;
            if (!(atomicOr(&S.row_flags[row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
            atomicExch(&S.counters[CNT_ERR], 1u);
            t2 = SS_DEAD;
          }
          p_state = t2;
          st[par[u]] = p_state;
        }
        uint32_t t = SS_DEAD;
        if (p_state != SS_DEAD) {
          t = fill_next(G, S, j, p_state, byte[u], true, rq);
          if (t == SS_CLAIMED) {  // ours to queue
            const uint32_t at = atomicAdd(&S.counters[CNT_LEVEL_REQ + L], 1u);
            if (at < req_half) {
              ulonglong2* e = S.cx.req2 + req_base + at;
              e->y = ((unsigned long long)j << 32) | ((unsigned long long)rq.frame1 << 24) | (rq.code << 8) | byte[u];
              __threadfence();
              st_release64(&e->x, (gen << 48) | ((unsigned long long)L << 40) | 1ull);
              t = SS_PENDING;
            } else {  // the depth's queue is full: nobody will compute it: give the row up, and let nobody wait
              diag(S, DIAG_QUEUE_FULL);
              const uint32_t row = __ldcg(&S.cx.jobs[j].row_acc) & 0x7FFFFFFFu;
              if (!(atomicOr(&S.row_flags[row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
              atomicExch(&S.counters[CNT_ERR], 1u);
              fill_publish(S, j, rq.frame1, rq.code, G.eq_of_byte[byte[u]], V_DEAD);
              t = SS_DEAD;
            }
          }
        }
        st[node[u]] = t;
        any_alive |= (t != SS_DEAD);
      }
    }
    __syncwarp();
    if (__any_sync(FULL, any_alive) && lane == 0) atomicOr(&S.counters[CNT_LEVEL_ALIVE + L], 1u);
    // ---- this CTA's part of the pass is done: its warps serve the queued transitions by ticket while
    // the other CTAs finish (see sweep_kernel)
    if (!pass_arrive(S, pass_phase)) return;
    const uint32_t all_passed = pass_phase * gridDim.x;
    const uint32_t takers = (expect_req > 4u * gridDim.x) ? (uint32_t)SWEEP_WARPS : 8u;
    bool have_ticket = false, gave_up = false;
    uint32_t ticket = 0;
    for (uint32_t polls = 0; warp < takers;) {
      if (!have_ticket) {
        if (lane == 0) ticket = atomicAdd(&S.counters[CNT_LEVEL_TAKEN + L], 1u);
        ticket = __shfl_sync(FULL, ticket, 0);
        have_ticket = true;
      }
      uint32_t passed = 0, queued = 0;
      if (lane == 0) {  // in this order: once all have passed, the number queued is final
        passed = ld_acquire(&S.counters[CNT_PASS_DONE]) >= all_passed ? 1u : 0u;
        queued = min(ld_acquire(&S.counters[CNT_LEVEL_REQ + L]), req_half);
      }
      passed = __shfl_sync(FULL, passed, 0);
      queued = __shfl_sync(FULL, queued, 0);
      if (ticket >= queued) {
        if (passed) break;
        if (++polls > poll_limit(S, 21)) {
          gave_up = true;
          if (lane == 0) diag(S, DIAG_WAIT_QUEUE);
        }
        if ((polls & 63u) == 0u && lane == 0 && ld_acquire(&S.counters[CNT_BAR_ERR])) gave_up = true;
        gave_up = __any_sync(FULL, gave_up);
        if (gave_up) break;
        __nanosleep(polls < 16u ? 40 : 200);
        continue;
      }
      polls = 0;
      unsigned long long rq0 = 0, rq1 = 0;
      if (lane == 0) {  // the entry is written right after its number was drawn: wait for it to land
        const unsigned long long want = (gen << 48) | ((unsigned long long)L << 40) | 1ull;
        for (uint32_t spin = 0; spin < poll_limit(S, 22); ++spin) {
          rq0 = ld_acquire64(&S.cx.req2[req_base + ticket].x);
          if (rq0 == want) break;
          rq0 = 0;
        }
        if (rq0) rq1 = __ldcg(&S.cx.req2[req_base + ticket].y);
      }
      rq0 = __shfl_sync(FULL, rq0, 0);
      rq1 = __shfl_sync(FULL, rq1, 0);
      have_ticket = false;
      if (rq0 == 0) {
        if (lane == 0) diag(S, DIAG_WAIT_QUEUE);
        gave_up = true;
        break;
      }
      const uint32_t j = (uint32_t)(rq1 >> 32), frame1 = (uint32_t)(rq1 >> 24) & 0xFFu, code = (uint32_t)(rq1 >> 8) & 0xFFFFu, pb = (uint32_t)rq1 & 0xFFu;
      const CtxJob cj = S.cx.jobs[j];
      uint32_t in_frame = frame1 ? frame1 - 1u : NOF;  // the frame whose sets the parent's items may name
      if (frame1 == 0u && code != CODE_CHART) {      // a set of the walk's own knows the frame it lives in
        const uint32_t salt = __ldcg(A.recs + ((size_t)j * A.cap + (code - LBASE)) * A.rec_words + AR_SALT);
        in_frame = salt ? salt - 1u : NOF;
      }
      const uint32_t r = wk.step(cj, j, code == CODE_CHART ? cj.m - 1u : code, in_frame, pb);
      uint32_t val = V_DEAD;
      if (r != T_DEAD) {
        val = r;
        // is the new set a root in its own right?  Looked up before anybody can see the set
        uint32_t fr = 0;
        if (lane == 0) fr = ld_acquire(A.recs + ((size_t)j * A.cap + r) * A.rec_words + AR_FRAME);
        fr = __shfl_sync(FULL, fr, 0);
        if (fr == 0u) resolve_frame(wk, cj, j, r);
      }
      if (lane == 0) fill_publish(S, j, frame1, code, G.eq_of_byte[pb], val);
    }
    if (gave_up && lane == 0) atomicExch(&S.counters[CNT_BAR_ERR], 1u);
    __shared__ uint32_t lvl_s[3];
    __syncthreads();
    if (threadIdx.x == 0) {
      lvl_s[0] = ld_acquire(&S.counters[CNT_LEVEL_ALIVE + L]);
      lvl_s[1] = ld_acquire(&S.counters[CNT_BAR_ERR]);
      lvl_s[2] = ld_acquire(&S.counters[CNT_LEVEL_REQ + L]);
    }
    __syncthreads();
    const bool alive = lvl_s[0] != 0u;
    if (lvl_s[1]) return;
    expect_req = lvl_s[2];
    last_level = L;
    if (!alive) break;  // nothing survives this depth in any job
  }
  {
    uint32_t abandoned = 0;
    if (lane == 0) abandoned = ld_acquire(&S.counters[CNT_BAR_ERR]);
    if (__shfl_sync(FULL, abandoned, 0) != 0u) return;  // the masks are zeroed when they are published
  }
  if (wk.big_mode) hset_clear_all(sw.w.hset, sw.w.hset_mask);
  if (lane == 0) {
    if (sw.n_computed | sw.n_created) {
      stat_add(S, CNT_STAT_CTX_TRANS, sw.n_computed);
      stat_add(S, CNT_STAT_CTX_STATES, sw.n_created);
      stat_add64(S, CNT_STAT_STEP_CYCLES, sw.cycles);
    }
    if (wk.n_frames) stat_add(S, CNT_STAT_FRAMES, wk.n_frames);
  }
  // ---- mask words: 32 tokens per warp pass, one ballot per word (token t is valid iff the node where its
  // bytes end was reached alive; EOS iff the chart is accepting)
  const uint32_t Wm = G.Wm;
  constexpr uint32_t MW = 6;
  const uint32_t visited_end = __ldg(&G.lvl_off[last_level + 1]);
  for (uint32_t c0 = gw; c0 < n_jobs * Wm; c0 += MW * GW) {
    uint32_t node[MW], s_[MW], dst[MW];
    bool valid[MW], eos_ok[MW];
#pragma unroll
    for (uint32_t u = 0; u < MW; ++u) {
      const uint32_t c = c0 + u * GW;
      valid[u] = c < n_jobs * Wm;
      const uint32_t tok = (c % Wm) * 32 + lane;
      node[u] = (valid[u] && tok < G.V) ? __ldg(&G.tok_node[tok]) : 0xFFFFFFFEu;
      dst[u] = (valid[u] && lane == 0) ? (uint32_t)__ldcg(&S.cx.jobs[__ldg(&S.cx.fjobs[c / Wm])].mrow) : 0u;
    }
#pragma unroll
    for (uint32_t u = 0; u < MW; ++u) {
      const uint32_t c = c0 + u * GW;
      s_[u] = SS_DEAD;
      eos_ok[u] = false;
      if (node[u] == 0xFFFFFFFFu) {  // a token without bytes: only EOS can be valid
        const uint32_t tok = (c % Wm) * 32 + lane;
        eos_ok[u] = ((int32_t)tok == G.eos) && (__ldcg(&S.cx.jobs[__ldg(&S.cx.fjobs[c / Wm])].row_acc) >> 31) != 0u;
      } else if (node[u] < visited_end) {
        s_[u] = __ldcg(S.cx.st32 + (size_t)(c / Wm) * stride + node[u]);
      }
    }
#pragma unroll
    for (uint32_t u = 0; u < MW; ++u) {
      if (!valid[u]) continue;  // (uniform)
      const uint32_t c = c0 + u * GW;
      const uint32_t ji = c / Wm, wd = c % Wm;
      uint32_t s = s_[u];
      if (s == SS_PENDING) {  // a leaf that waited for a transition: its parent is final by now
        const uint32_t j = __ldg(&S.cx.fjobs[ji]);
        const uint32_t* st = S.cx.st32 + (size_t)ji * stride;
        const uint32_t start = __ldcg(&S.cx.jobs[j].pad[0]) ? ((1u << 16) | RBASE) : CODE_CHART;
        const uint32_t p = __ldg(&G.parent[node[u]]);
        const uint32_t p_state = (p == 0) ? start : __ldcg(st + p);
        const uint32_t nbyte = __ldg(&G.node_byte[node[u]]);
        FillReq rq;
        uint32_t t2 = (p_state == SS_DEAD || p_state == SS_PENDING) ? SS_DEAD : fill_next(G, S, j, p_state, nbyte, false, rq);
        for (uint32_t spin = 0; t2 == SS_PENDING && spin < poll_limit(S, 21); ++spin) {
          __nanosleep(40);
          t2 = fill_next(G, S, j, p_state, nbyte, false, rq);
        }
        if (t2 == SS_PENDING || p_state == SS_PENDING) {
          diag(S, DIAG_WAIT_VALUE);
          const uint32_t row = __ldcg(&S.cx.jobs[j].row_acc) & 0x7FFFFFFFu;
          if (!(atomicOr(&S.row_flags[row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
          t2 = SS_DEAD;
        }
        s = t2;
      }
      const uint32_t word = __ballot_sync(FULL, s != SS_DEAD || eos_ok[u]);
      if (lane == 0) S.mask_rows[(size_t)dst[u] * Wm + wd] = word;
    }
  }
}

// ===================================================================================== launchers

cudaError_t configure_walk_kernels() {
  return cudaFuncSetAttribute((const void*)fill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
}

void launch_fill(const GrammarDev& G, const StateDev& S, int sweep_grid, cudaStream_t st, cudaEvent_t before_roots,
                 cudaEvent_t after_roots, cudaEvent_t before_sweep, cudaEvent_t after_sweep) {
  launch_plan(G, S, st);
  if (!S.rt.on) {
    // without the cache of context-independent entries every row is swept from its chart's last set
    if (before_sweep) cudaEventRecord(before_sweep, st);
    launch_sweep(G, S, sweep_grid, st);
    if (after_sweep) cudaEventRecord(after_sweep, st);
    launch_publish(S, st);
    return;
  }
  if (before_roots) cudaEventRecord(before_roots, st);
  const unsigned job_blocks = (unsigned)std::min<uint32_t>((S.B + ROOT_WARPS - 1) / ROOT_WARPS, 296u);
  pending_kernel<<<1, 32, 0, st>>>(S);
  root_kernel<<<job_blocks, ROOT_WARPS * 32, 0, st>>>(G, S);
  if (S.rt.on) {
    // the sweep of this fill's new roots sees them as the rows of a state of its own
    StateDev R = S;
    R.ctx_mode = 1;
    R.arena = S.rt.charts;
    R.row_chart = S.rt.rj_chart;
    R.row_mask = S.rt.rj_mask;
    R.row_flags = S.rt.rj_flags;
    R.jobs = S.rt.rj_jobs;
    R.counters = S.rt.counters;
    R.mask_rows = S.rt.ci_rows;
    launch_sweep(G, R, sweep_grid, st);
    collect_kernel<<<S.B, COLLECT_THREADS, 0, st>>>(G, S);
  }
  if (after_roots) cudaEventRecord(after_roots, st);
  if (before_sweep) cudaEventRecord(before_sweep, st);
  job_setup_kernel<<<std::min<uint32_t>(S.B, 296u), 256, 0, st>>>(G, S);
  {  // (launched cooperatively: its thread blocks wait for one another between the trie's depths)
    GrammarDev g = G;
    StateDev s = S;
    void* args[] = {&g, &s};
    cudaLaunchCooperativeKernel((const void*)fill_kernel, dim3((unsigned)sweep_grid), dim3(SWEEP_WARPS * 32), args, S.au.smem_bytes, st);
  }
  if (after_sweep) cudaEventRecord(after_sweep, st);
  launch_publish(S, st);
}

}  // namespace fmt
