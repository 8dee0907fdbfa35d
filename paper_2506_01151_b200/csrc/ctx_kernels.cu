// The mask fill in two parts (Section 4.3 of the paper: tokens whose validity does not depend on the
// context are looked up, only the context-dependent ones are checked against the parser state).
//
//   root_kernel      per computed row: its chart's last set with anonymous origins (a "root") is
//                    looked up in, or added to, the directory of roots
//   sweep_kernel     (kernels.cu, root mode) the trie sweep of every new root, once for good
//   collect_kernel   turns a finished root sweep into the root's frontier list and region of sets
//   ctx_init_kernel  starts every job's mask row from its root's context-independent mask
//   ctx_kernel       the context-dependent walk: from each frontier node on, Earley steps against the
//                    row's own chart (Section 3.2), memoised per job, spread over the grid by a queue
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
__device__ __forceinline__ uint32_t ctx_poll_limit(const StateDev& S, uint32_t dflt) {
  return 1u << (S.poll_limit_shift ? S.poll_limit_shift : dflt);
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
      cj.fr_off = cj.fr_n = cj.st_off = 0;
      cj.mrow = S.row_mask[row];
      cj.pad[0] = cj.pad[1] = 0;
      S.cx.jobs[j] = cj;
    }
  }
}

// ===================================================================================== collect
//
// After the root sweep: one CTA per swept root keeps what later fills need.  The sweep left, per trie
// node, the set the node leads to (or dead / context-dependent) and, per set, its items.  Kept are
// the frontier (nodes marked context-dependent, with the set of their parent), in node order, and
// the items of every set (the walk of a row reads them with its own bindings); the transitions are
// not needed again: the trie has been swept for good.

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
      fo = atomicAdd(&R.tops[TOP_FRONTIER], fr_total);
      so = atomicAdd(&R.tops[TOP_STATES], nst);
      io = atomicAdd(&R.tops[TOP_ITEMS], it_total);
      to = atomicAdd(&R.tops[TOP_TRANS], tr_total);
      if (fo > R.fr_cap || fr_total > R.fr_cap - fo || so > R.st_cap || nst > R.st_cap - so || io > R.it_cap || it_total > R.it_cap - io ||
          to > R.tr_cap || tr_total > R.tr_cap - to)
        f = 1u;
    }
    sh[0] = fo, sh[1] = so, sh[2] = io, sh[3] = f, sh[4] = to;
  }
  if (threadIdx.x < 256) rep_byte[threadIdx.x] = 0u;
  __syncthreads();
  if (threadIdx.x < 256) rep_byte[G.eq_of_byte[threadIdx.x]] = (uint8_t)threadIdx.x;  // any byte of the class will do
  __syncthreads();
  const uint32_t fr_off = sh[0], st_off = sh[1], it_off = sh[2], tr_off = sh[4];
  failed = sh[3] != 0u;
  if (!failed) {
    // ---- pass 2: the frontier in node order
    uint32_t done = 0;
    for (uint32_t base = 1; base < visited_end; base += blockDim.x) {
      const uint32_t node = base + threadIdx.x;
      uint32_t ps = 0;
      const bool is_f = node < visited_end && frontier_at(node, ps);
      uint32_t tile;
      const uint32_t at = block_scan(is_f ? 1u : 0u, sums, tile);
      if (is_f) R.frontier[fr_off + done + at] = make_uint2(node, ps | ((uint32_t)G.eq_of_byte[G.node_byte[node]] << 16));
      done += tile;
    }
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
    info[RI_FR_OFF] = fr_off;
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

// ===================================================================================== walk: set-up
//
// Every job's mask row starts as its root's context-independent mask (or empty), plus the EOS bit of
// an accepting chart; block 0 also lists the work: the frontier of every job in chunks of 32 entries,
// and gives every job with a usable root its frame 0.  A job without one starts at the trie's first
// level with the chart's own last set.

__global__ void __launch_bounds__(1024) ctx_init_kernel(GrammarDev G, StateDev S) {
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  const RootDev& R = S.rt;
  const uint32_t Wm = G.Wm;
  auto ready = [&](const CtxJob& cj) { return cj.root != ROOT_NONE && __ldcg(R.info + (size_t)cj.root * RI_WORDS + RI_STATUS) == ROOT_READY; };
  for (uint32_t j = blockIdx.x; j < n_jobs; j += gridDim.x) {
    const CtxJob cj = S.cx.jobs[j];
    const bool use = ready(cj);
    const uint32_t* src = use ? R.ci_rows + (size_t)cj.root * Wm : nullptr;
    uint32_t* dst = S.mask_rows + (size_t)cj.mrow * Wm;
    const bool acc = (cj.row_acc >> 31) != 0u && G.eos >= 0;
    for (uint32_t w = threadIdx.x; w < Wm; w += blockDim.x) {
      uint32_t v = src ? src[w] : 0u;
      if (acc && w == ((uint32_t)G.eos >> 5)) v |= 1u << ((uint32_t)G.eos & 31u);
      dst[w] = v;
    }
    // frame 0: the job's own root, its placeholders bound as root_kernel found them
    const uint32_t* info = R.info + (size_t)(use ? cj.root : 0u) * RI_WORDS;
    if (threadIdx.x == 0) {
      Frame f;
      f.root = cj.root, f.P = cj.P, f.n = use ? info[RI_NSTATES] : 0u;
      f.st_off = use ? info[RI_ST_OFF] : 0u, f.tr_off = use ? info[RI_TR_OFF] : 0u, f.pad0 = f.pad1 = f.pad2 = 0u;
      S.cx.frames[(size_t)j * MAXF] = f;
      S.cx.frame_ctr[j] = use ? 1u : 0u;
    }
    if (use)
      for (uint32_t i = threadIdx.x; i < cj.P && i < R.max_ph; i += blockDim.x)
        S.cx.fbind[(size_t)j * MAXF * R.max_ph + i] = S.cx.bind[(size_t)j * R.max_ph + i];
  }
  if (blockIdx.x != 0) return;
  __shared__ uint32_t sums[33];
  uint32_t run = 0;
  for (uint32_t base = 0; base < n_jobs; base += blockDim.x) {
    const uint32_t j = base + threadIdx.x;
    uint32_t chunks = 0;
    if (j < n_jobs) {
      CtxJob cj = S.cx.jobs[j];
      const bool use = ready(cj);
      const uint32_t* info = R.info + (size_t)(use ? cj.root : 0u) * RI_WORDS;
      uint32_t fr_off, fr_n, st_off = 0;
      if (use) {
        fr_off = info[RI_FR_OFF], fr_n = info[RI_FR_N], st_off = info[RI_ST_OFF];
        stat_add(S, CNT_STAT_JOBS_ROOT, 1u);
      } else {
        fr_off = G.lvl_off[1], fr_n = G.lvl_off[2] - G.lvl_off[1];
        stat_add(S, CNT_STAT_JOBS_PLAIN, 1u);
      }
      S.cx.jobs[j].fr_off = fr_off;
      S.cx.jobs[j].fr_n = fr_n;
      S.cx.jobs[j].st_off = st_off;
      S.cx.jobs[j].pad[0] = use ? 1u : 0u;
      S.au.n_states[j] = 0u;
      chunks = (fr_n + 31u) / 32u;
    }
    uint32_t tile;
    const uint32_t at = block_scan(chunks, sums, tile);
    if (j < n_jobs) S.cx.chunk_off[j] = run + at;
    run += tile;
  }
  if (threadIdx.x == 0) {
    S.cx.chunk_off[n_jobs] = run;
    S.cx.qctr[Q_TAIL] = 0u;
    S.cx.qctr[Q_HEAD] = 0u;
    S.cx.qctr[Q_OUT] = run;
    S.cx.qctr[Q_CHUNK] = 0u;
    S.cx.qctr[Q_CHUNKS] = run;
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
constexpr uint32_t STACK_NODES = 4096;                      // nodes a warp may hold for itself (node, set code | job << 16, frame)
constexpr uint32_t STACK_WORDS = 3u * STACK_NODES;
constexpr uint32_t SHARE_ABOVE = 6, SHARE_N = 32;           // a warp holding more nodes than this hands all but 4 (at most 32) to the queue
constexpr uint32_t V_DEAD = 0xFFFFu, V_PEND = 0xFFFEu;      // values of a remembered transition (16 bits)
constexpr uint32_t CODE_CHART = 0xFFFFu;                    // "parent set" of a job without a root: the chart's last set

struct Walker {
  const GrammarDev& G;
  const StateDev& S;
  SweepWarp& sw;
  uint32_t* big;
  bool big_mode = false;
  uint32_t n_frontier = 0, n_tasks = 0, n_nodes = 0, n_frames = 0;
  // Nodes waiting to be expanded by this warp: a stack at the top of the warp's large scratch area
  // (the sets under construction use the part below).  Entry: node, set code | job << 16.
  uint32_t held = 0;
  __device__ __forceinline__ uint32_t* stack() const { return big + (S.big_arena_items - STACK_WORDS); }

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
    const uint32_t* pitems;
    uint32_t plen;
    v(pcode, pitems, plen);
    uint32_t r = sw.step(J, v, pitems, plen, pcode, byte, !big_mode);
    if (r == T_FAIL && !big_mode) {  // a set outgrew the shared-memory scratch: use the large area from now on
      big_mode = true;
      hset_clear_all(sw.w.hset, sw.w.hset_mask);
      clear_nt(G, sw.w);
      sw.w.cur = big;
      sw.w.cur_cap = S.big_arena_items - STACK_WORDS;
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
  // the tokens whose bytes end at `node` are valid
  __device__ __forceinline__ void mark_tokens(const CtxJob& cj, uint32_t node) const {
    uint32_t* row = S.mask_rows + (size_t)cj.mrow * G.Wm;
    for (uint32_t i = __ldg(&G.tok_off[node]), e = __ldg(&G.tok_off[node + 1]); i < e; ++i) {
      const uint32_t t = __ldg(&G.tok_ids[i]);
      atomicOr(&row[t >> 5], 1u << (t & 31u));
    }
  }
  // The nodes of the lanes with `want` (alive, reached in set `code`, with children) go onto this warp's stack.
  __device__ void keep(const CtxJob& cj, uint32_t j, bool want, uint32_t node, uint32_t code, uint32_t frame) {
    const uint32_t lane = lane_id();
    const uint32_t wb = __ballot_sync(FULL, want);
    if (!wb) return;
    const uint32_t k = held + __popc(wb & ((1u << lane) - 1u));
    bool gone = false;
    if (want) {
      if (k < STACK_NODES) {
        uint32_t* st = stack();
        st[3u * k] = node;
        st[3u * k + 1u] = code | (j << 16);
        st[3u * k + 2u] = frame;
      } else {
        gone = true;
      }
    }
    held = min(held + __popc(wb), STACK_NODES);
    __syncwarp();
    if (__any_sync(FULL, gone)) {  // (the queue was full and the stack is, too)
      if (lane == 0) diag(S, DIAG_QUEUE_FULL);
      break_row(job(cj, j));
    }
  }
  // A warp that holds many nodes hands the oldest ones (the largest subtrees) to the queue.
  __device__ void share() {
    if (held <= SHARE_ABOVE) return;
    const uint32_t lane = lane_id();
    uint32_t base = 0, fit = 0;
    const uint32_t give = min(SHARE_N, held - 4u);
    if (lane == 0) {
      if (ld_acquire(&S.cx.qctr[Q_TAIL]) + give <= S.cx.q_cap) {
        base = atomicAdd(&S.cx.qctr[Q_TAIL], give);
        fit = base >= S.cx.q_cap ? 0u : min(give, S.cx.q_cap - base);
        atomicAdd(&S.cx.qctr[Q_OUT], fit);  // (before this warp reports its own unit done)
      }
    }
    base = __shfl_sync(FULL, base, 0);
    fit = __shfl_sync(FULL, fit, 0);
    if (fit == 0) return;
    uint32_t* st = stack();
    if (lane < fit) {
      uint4* e = S.cx.queue + base + lane;
      const uint32_t node = st[3u * lane], cj_ = st[3u * lane + 1u], fr_ = st[3u * lane + 2u];
      e->x = node, e->y = (cj_ & 0xFFFFu) | (fr_ << 16), e->z = cj_ >> 16;
      __threadfence();
      st_release32(&e->w, (S.gen_ctx << 16) | 1u);
    }
    __syncwarp();
    for (uint32_t i0 = 0; i0 + fit < held; i0 += 32) {  // close the gap
      const uint32_t i = i0 + lane;
      uint32_t a = 0, b = 0, c = 0;
      if (i + fit < held) a = st[3u * (i + fit)], b = st[3u * (i + fit) + 1u], c = st[3u * (i + fit) + 2u];
      __syncwarp();
      if (i + fit < held) st[3u * i] = a, st[3u * i + 1u] = b, st[3u * i + 2u] = c;
      __syncwarp();
    }
    held -= fit;
    n_tasks += fit;
  }
};

// The set that job j reaches from the set `code` of `frame` (or, with CODE_CHART and no frame, from
// the chart's last set) on the byte class `eq`, for the lanes with `valid`: looked up in the job's
// table of such transitions, computed by this warp if nobody has yet (one Earley step against the
// row's chart).  Returns the walk's id of the set, or V_DEAD.  Called by all lanes.
__device__ uint32_t ctx_transition(Walker& wk, const CtxJob& cj, uint32_t j, bool valid, uint32_t frame, uint32_t code, uint32_t eq,
                                   uint32_t byte) {
  const StateDev& S = wk.S;
  const uint32_t lane = lane_id();
  const unsigned long long key = ((unsigned long long)((frame + 1u) & 0xFFu) << 24) | (code << 8) | eq;  // 32 bits
  const unsigned long long gen = S.gen_ctx & 0xFFFFu;
  unsigned long long* tab = S.cx.ctab + (size_t)j * CT_SLOTS;
  // ---- one lane per distinct key asks the table
  const uint32_t peers = __match_any_sync(FULL, valid ? key : ((1ull << 40) | lane));  // (a key has 32 bits: idle lanes match nobody)
  const bool leader = valid && (uint32_t)(__ffs(peers) - 1) == lane;
  uint32_t val = V_PEND;
  int slot = -1;       // >= 0: the slot that holds (or will hold) the value
  bool mine = false;   // this lane computes the value
  if (leader) {
    uint32_t s = (mix32((uint32_t)key) & (CT_SLOTS - 1));
    for (uint32_t probe = 0; probe < 64; ++probe) {
      unsigned long long v = ld_acquire64(tab + s);
      if ((v >> 48) != gen) {  // left by an earlier fill: free
        const unsigned long long nv = (gen << 48) | (key << 16) | V_PEND;
        const unsigned long long old = atomicCAS(tab + s, v, nv);
        if (old == v) {
          slot = (int)s;
          mine = true;
          break;
        }
        v = old;
        if ((v >> 48) != gen) {
          --probe;  // (taken and released again: look once more)
          continue;
        }
      }
      if (((v >> 16) & 0xFFFFFFFFull) == key) {
        slot = (int)s;
        val = (uint32_t)v & 0xFFFFu;
        break;
      }
      s = (s + 1u) & (CT_SLOTS - 1);
    }
    if (slot < 0) mine = true;  // no room in the table: compute it all the same, it just is not remembered
  }
  // ---- the warp computes what its lanes have claimed, one transition at a time
  uint32_t todo = __ballot_sync(FULL, mine);
  while (todo) {
    const int src = __ffs(todo) - 1;
    todo &= todo - 1;
    const uint32_t scode = __shfl_sync(FULL, code, src), sbyte = __shfl_sync(FULL, byte, src), sframe = __shfl_sync(FULL, frame, src);
    const uint32_t r = wk.step(cj, j, scode == CODE_CHART ? cj.m - 1u : scode, sframe, sbyte);
    if (lane == 0) diag(S, 11);
    if ((int)lane == src) {
      val = (r == T_DEAD) ? V_DEAD : r;
      if (slot >= 0) st_release64(tab + slot, (gen << 48) | (key << 16) | val);
    }
  }
  // ---- a value somebody else is computing: wait for it (the other warp is at it, it waits for nothing)
  if (leader && val == V_PEND) {
    const uint32_t limit = ctx_poll_limit(S, 22);
    for (uint32_t spin = 0; spin < limit; ++spin) {
      const unsigned long long v = ld_acquire64(tab + slot);
      val = (uint32_t)v & 0xFFFFu;
      if (val != V_PEND) break;
      __nanosleep(100);
    }
    if (val == V_PEND) {
      diag(S, DIAG_WAIT_VALUE);
      atomicExch(&S.counters[CNT_BAR_ERR], 1u);
      val = V_DEAD;
    }
  }
  return __shfl_sync(FULL, val, __ffs(peers) - 1);
}

// A chunk of 32 frontier entries of job j, one per lane: nodes reached alive mark their tokens and
// are kept for expansion if they have children.
__device__ void walk_chunk(Walker& wk, uint32_t j, uint32_t e0) {
  const GrammarDev& G = wk.G;
  const StateDev& S = wk.S;
  const uint32_t lane = lane_id();
  const CtxJob cj = S.cx.jobs[j];
  const bool use_root = cj.pad[0] != 0u;
  const uint32_t e = e0 + lane;
  const bool valid = e < cj.fr_n;
  uint32_t node = 0, code = CODE_CHART, eq = 0;
  const uint32_t frame = use_root ? 0u : NOF;  // (frame 0 is the job's own root)
  if (valid) {
    if (use_root) {
      const uint2 fe = __ldg(S.rt.frontier + cj.fr_off + e);
      node = fe.x, code = RBASE + (fe.y & 0xFFFFu), eq = fe.y >> 16;
    } else {
      node = cj.fr_off + e;
      eq = G.eq_of_byte[__ldg(&G.node_byte[node])];
    }
  }
  const uint32_t byte = valid ? __ldg(&G.node_byte[node]) : 0u;
  const uint32_t val = ctx_transition(wk, cj, j, valid, frame, code, eq, byte);
  const bool alive = valid && val != V_DEAD;
  if (alive) wk.mark_tokens(cj, node);
  const bool kids = alive && __ldg(&G.child_off[node + 1]) > __ldg(&G.child_off[node]);
  wk.keep(cj, j, kids, node, LBASE + val, NOF);  // (a set of the walk's own knows the frame it lives in)
  wk.n_frontier += __popc(__ballot_sync(FULL, valid));
}

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
  uint32_t result = NOFRAME, why = 15;
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
    why = 13;
    if (ok) {
      why = 15;
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
        why = 14;
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
              why = 0;
              ++wk.n_frames;
            }
          }
        }
      }
    }
  }
  if (lane == 0 && why) diag(S, why);
  uint32_t old = 0;
  if (lane == 0) old = atomicCAS(rec + AR_FRAME, 0u, result);
  old = __shfl_sync(FULL, old, 0);
  return old != 0u ? old : result;  // (another warp may have looked the same set up meanwhile: use its answer)
}

// ---- What a root's region makes of the subtree of a node (see RootDev::mkey): computed once, by table
// look-ups alone, by the first warp that needs it.  The warp's large scratch area holds the work:
constexpr uint32_t MEMO_TOK = 24u * 1024u;   // tokens found                       [0, MEMO_TOK)
constexpr uint32_t MEMO_FR = 4096u;          // frontier entries (two words each)  [MEMO_TOK, + 2 * MEMO_FR)
constexpr uint32_t MEMO_STACK = 4096u;       // nodes to visit (two words each)    [.., + 2 * MEMO_STACK)
static_assert(MEMO_TOK + 2 * MEMO_FR + 2 * MEMO_STACK + STACK_WORDS <= 65536, "the large scratch area is 64 Ki words");

// Returns entry + 1, or 0 when there is no entry to use (another warp is computing it, or it does not fit).
__device__ uint32_t memo_get(Walker& wk, uint32_t rid, uint32_t tr_off, uint32_t node) {
  const GrammarDev& G = wk.G;
  const StateDev& S = wk.S;
  const RootDev& R = S.rt;
  const uint32_t lane = lane_id();
  const unsigned long long key = ((unsigned long long)(rid + 1u) << 32) | node;
  uint32_t slot = (mix32(node) ^ mix32(rid * 0x9E3779B9u + 1u)) & R.m_mask;
  uint32_t state = 0;  // 1: ours to compute (slot), 2: there (val), 3: none
  uint32_t val = 0;
  if (lane == 0) {
    state = 3;
    for (uint32_t probe = 0; probe < 32; ++probe) {
      unsigned long long k = ld_acquire64(R.mkey + slot);
      if (k == 0ull) {
        k = atomicCAS(R.mkey + slot, 0ull, key);
        if (k == 0ull) {
          state = 1;
          break;
        }
      }
      if (k == key) {
        val = ld_acquire(R.mval + slot);
        state = 2;
        break;
      }
      slot = (slot + 1u) & R.m_mask;
    }
  }
  state = __shfl_sync(FULL, state, 0);
  val = __shfl_sync(FULL, val, 0);
  slot = __shfl_sync(FULL, slot, 0);
  if (state == 2) return val;
  if (state != 1 || S.big_arena_items < 65536u) return 0;
  // ---- depth first through the subtree, in the region's transition table
  uint32_t* tok = wk.big;
  uint32_t* fr = wk.big + MEMO_TOK;
  uint32_t* stk = fr + 2 * MEMO_FR;
  uint32_t n_tok = 0, n_fr = 0, n_stk = 1;
  bool ok = true;
  if (lane == 0) stk[0] = node, stk[1] = 0u;  // the walk stands in the root set
  __syncwarp();
  while (n_stk && ok) {
    --n_stk;
    const uint32_t nd = stk[2u * n_stk], k = stk[2u * n_stk + 1u];
    __syncwarp();
    const uint16_t* row = R.trans + tr_off + (size_t)k * G.n_eq;
    const uint32_t c0 = __ldg(&G.child_off[nd]), c1 = __ldg(&G.child_off[nd + 1]);
    for (uint32_t base = c0; base < c1 && ok; base += 32) {
      const uint32_t c = base + lane;
      const bool valid = c < c1;
      const uint32_t eq = valid ? (uint32_t)G.eq_of_byte[__ldg(&G.node_byte[c])] : 0u;
      const uint32_t t16 = valid ? (uint32_t)__ldg(row + eq) : (uint32_t)R_DEAD;
      const bool alive = t16 < R_CTX, ctx = t16 == R_CTX;
      // the tokens that end at the children reached alive
      const uint32_t t0 = alive ? __ldg(&G.tok_off[c]) : 0u, cnt = alive ? __ldg(&G.tok_off[c + 1]) - t0 : 0u;
      uint32_t incl = cnt;
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(FULL, incl, d);
        if ((int)lane >= d) incl += t;
      }
      const uint32_t total = __shfl_sync(FULL, incl, 31);
      const uint32_t fb = __ballot_sync(FULL, ctx);
      const bool kids = alive && __ldg(&G.child_off[c + 1]) > __ldg(&G.child_off[c]);
      const uint32_t kb = __ballot_sync(FULL, kids);
      if (n_tok + total > MEMO_TOK || n_fr + __popc(fb) > MEMO_FR || n_stk + __popc(kb) > MEMO_STACK) {
        ok = false;
        break;
      }
      for (uint32_t i = 0; i < cnt; ++i) tok[n_tok + incl - cnt + i] = __ldg(&G.tok_ids[t0 + i]);
      if (ctx) {
        const uint32_t at = n_fr + __popc(fb & ((1u << lane) - 1u));
        fr[2u * at] = c, fr[2u * at + 1u] = k | (eq << 16);
      }
      if (kids) {
        const uint32_t at = n_stk + __popc(kb & ((1u << lane) - 1u));
        stk[2u * at] = c, stk[2u * at + 1u] = t16;
      }
      n_tok += total, n_fr += __popc(fb), n_stk += __popc(kb);
      __syncwarp();
    }
  }
  // ---- keep it
  uint32_t ent = 0;
  if (ok) {
    const uint32_t words = n_tok + 2u * n_fr;
    uint32_t e = 0, d = 0;
    if (lane == 0) {
      e = atomicAdd(&R.tops[TOP_MENT], 1u);
      d = atomicAdd(&R.tops[TOP_MDATA], words);
      if (e >= R.me_cap || d > R.md_cap || words > R.md_cap - d) e = 0xffffffffu;
    }
    e = __shfl_sync(FULL, e, 0);
    d = __shfl_sync(FULL, d, 0);
    if (e != 0xffffffffu) {
      for (uint32_t i = lane; i < n_tok; i += 32) R.mdata[d + i] = tok[i];
      for (uint32_t i = lane; i < 2u * n_fr; i += 32) R.mdata[d + n_tok + i] = fr[i];
      if (lane == 0) R.ment[e] = make_uint4(d, n_tok, n_fr, 0u);
      __syncwarp();
      __threadfence();
      ent = e + 1u;
      if (lane == 0) st_release32(R.mval + slot, ent);
    }
  }
  return ent;
}

// Job j stands at `node` in the root set of frame `fi`: mark what the region alone decides below the
// node and keep the nodes where the chart is needed again.
__device__ void memo_apply(Walker& wk, const CtxJob& cj, uint32_t j, uint32_t frame, uint32_t ent) {
  const GrammarDev& G = wk.G;
  const StateDev& S = wk.S;
  const RootDev& R = S.rt;
  const uint32_t lane = lane_id();
  const uint4 e = __ldcg(R.ment + ent - 1u);
  const uint32_t* tok = R.mdata + e.x;
  const uint32_t* fr = tok + e.y;
  uint32_t* row = S.mask_rows + (size_t)cj.mrow * G.Wm;
  for (uint32_t i = lane; i < e.y; i += 32) {
    const uint32_t t = __ldcg(tok + i);
    atomicOr(&row[t >> 5], 1u << (t & 31u));
  }
  for (uint32_t base = 0; base < e.z; base += 32) {
    const uint32_t i = base + lane;
    const bool valid = i < e.z;
    const uint32_t node = valid ? __ldcg(fr + 2u * i) : 0u, ke = valid ? __ldcg(fr + 2u * i + 1u) : 0u;
    const uint32_t byte = valid ? __ldg(&G.node_byte[node]) : 0u;
    const uint32_t val = ctx_transition(wk, cj, j, valid, frame, RBASE + (ke & 0xFFFFu), ke >> 16, byte);
    const bool alive = valid && val != V_DEAD;
    if (alive) wk.mark_tokens(cj, node);
    const bool kids = alive && __ldg(&G.child_off[node + 1]) > __ldg(&G.child_off[node]);
    wk.keep(cj, j, kids, node, LBASE + val, NOF);
  }
  wk.n_frontier += e.z;
}

// The children of `node`, which job j reached in the set `code` (of `frame`, if it is a frame's set).
__device__ void walk_expand(Walker& wk, uint32_t j, uint32_t node, uint32_t code, uint32_t frame) {
  const GrammarDev& G = wk.G;
  const StateDev& S = wk.S;
  const AutoDev& A = S.au;
  const uint32_t lane = lane_id();
  const CtxJob cj = S.cx.jobs[j];
  ++wk.n_nodes;
  if (code < RBASE) {  // a set this walk made: it lives in some frame, and may be a root in its own right
    const uint32_t id = code - LBASE;
    const uint32_t* rec = A.recs + ((size_t)j * A.cap + id) * A.rec_words;
    uint32_t fr = 0;  // (one lane looks, all lanes act on what it saw: another warp may be writing the answer just now)
    if (lane == 0) fr = ld_acquire(rec + AR_FRAME);
    fr = __shfl_sync(FULL, fr, 0);
    if (fr == 0u) fr = resolve_frame(wk, cj, j, id);
    if (fr != NOFRAME) {
      frame = fr - 1u;
      code = RBASE;  // set 0 of the frame it opens
      if (!wk.big_mode) {  // (the look-up below works in the warp's large scratch area: not while sets are built there)
        const Frame* f = S.cx.frames + (size_t)j * MAXF + frame;
        const uint32_t ent = memo_get(wk, __ldcg(&f->root), __ldcg(&f->tr_off), node);
        if (ent) {
          if (lane == 0) diag(S, 8);
          memo_apply(wk, cj, j, frame, ent);
          return;
        }
      }
    } else {
      const uint32_t salt = __ldcg(rec + AR_SALT);
      frame = salt ? salt - 1u : NOF;
    }
  }
  const uint32_t c0 = __ldg(&G.child_off[node]), c1 = __ldg(&G.child_off[node + 1]);
  if (code >= RBASE) {
    // ---- a frame's set: one table look-up per child; only context-dependent transitions cost a step
    if (lane == 0) diag(S, 9);
    const Frame* f = S.cx.frames + (size_t)j * MAXF + frame;
    const uint16_t* row = S.rt.trans + __ldcg(&f->tr_off) + (size_t)(code - RBASE) * G.n_eq;
    for (uint32_t base = c0; base < c1; base += 32) {
      const uint32_t c = base + lane;
      const bool valid = c < c1;
      const uint32_t byte = valid ? __ldg(&G.node_byte[c]) : 0u;
      const uint32_t eq = G.eq_of_byte[byte];
      const uint32_t t16 = valid ? (uint32_t)__ldg(row + eq) : (uint32_t)R_DEAD;
      const bool is_ctx = valid && t16 == R_CTX;
      uint32_t ccode = RBASE + t16;
      bool alive = valid && t16 < R_CTX;
      if (__any_sync(FULL, is_ctx)) {
        const uint32_t val = ctx_transition(wk, cj, j, is_ctx, frame, code, eq, byte);
        if (is_ctx && val != V_DEAD) alive = true, ccode = LBASE + val;
      }
      if (alive) wk.mark_tokens(cj, c);
      const bool kids = alive && __ldg(&G.child_off[c + 1]) > __ldg(&G.child_off[c]);
      wk.keep(cj, j, kids, c, ccode, frame);
    }
    return;
  }
  // ---- a set of the walk's own: its transitions are Earley steps, remembered in its record
  if (lane == 0) diag(S, 10);
  const uint32_t state = code - LBASE;
  uint32_t* rec = A.recs + ((size_t)j * A.cap + state) * A.rec_words;
  for (uint32_t base = c0; base < c1; base += 32) {
    const uint32_t c = base + lane;
    const bool valid = c < c1;
    const uint32_t byte = valid ? __ldg(&G.node_byte[c]) : 0u;
    uint32_t t = T_DEAD;
    uint32_t* slot = nullptr;
    bool mine = false;
    // one 256-bit test rejects most bytes without touching the transition table
    if (valid && ((__ldcg(rec + AR_SCAN + (byte >> 5)) >> (byte & 31u)) & 1u)) {
      slot = rec + AR_TRANS + G.eq_of_byte[byte];
      t = ld_acquire(slot);
      if (t == T_UNKNOWN) {
        t = atomicCAS(slot, T_UNKNOWN, T_PENDING);
        if (t == T_UNKNOWN) mine = true, t = T_PENDING;
      }
    }
    uint32_t todo = __ballot_sync(FULL, mine);
    while (todo) {
      const int src = __ffs(todo) - 1;
      todo &= todo - 1;
      const uint32_t sbyte = __shfl_sync(FULL, byte, src);
      const uint32_t r = wk.step(cj, j, code, frame, sbyte);
      if (lane == 0) diag(S, 12);
      if ((int)lane == src) {
        t = r;
        st_release32(slot, r);
      }
    }
    if (t == T_PENDING) {  // another lane or warp claimed it before this lane asked
      const uint32_t limit = ctx_poll_limit(S, 22);
      for (uint32_t spin = 0; spin < limit; ++spin) {
        t = ld_acquire(slot);
        if (t != T_PENDING) break;
        __nanosleep(100);
      }
      if (t == T_PENDING) {
        diag(S, DIAG_WAIT_VALUE);
        atomicExch(&S.counters[CNT_BAR_ERR], 1u);
        t = T_DEAD;
      }
    }
    const bool alive = valid && t != T_DEAD;
    if (alive) wk.mark_tokens(cj, c);
    const bool kids = alive && __ldg(&G.child_off[c + 1]) > __ldg(&G.child_off[c]);
    wk.keep(cj, j, kids, c, LBASE + t, NOF);
  }
}

// The walk of all jobs of a fill.  Work units: first the chunks of frontier entries, handed out by
// a counter; then nodes drawn from a queue.  A warp expands the nodes of its unit depth first from a
// stack of its own and hands nodes to the queue only when it holds many, so that most nodes cost no
// atomic operation; a warp that finds the queue empty waits for either a new entry or the count of
// unfinished units to reach zero.  No unit ever waits for another unit, only for a single Earley step
// that another warp is computing, so every wait ends; all the same each is a poll with a limit that
// flags an error instead of hanging.
__global__ void __launch_bounds__(SWEEP_WARPS * 32, 1) ctx_kernel(GrammarDev Gg, StateDev S) {
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  if (n_jobs == 0) return;
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
  uint32_t* q = S.cx.qctr;
  const uint32_t n_chunks = q[Q_CHUNKS];
  const uint32_t tag = (S.gen_ctx << 16) | 1u;
  const uint32_t limit = ctx_poll_limit(S, 22);
  bool chunks_left = true, abandoned = false;

  for (;;) {
    bool have = false;
    if (chunks_left) {  // ---- a chunk of some job's frontier
      uint32_t c = 0;
      if (lane == 0) c = atomicAdd(&q[Q_CHUNK], 1u);
      c = __shfl_sync(FULL, c, 0);
      if (c < n_chunks) {
        uint32_t lo = 0, hi = n_jobs;  // the job whose chunks include c: chunk_off[lo] <= c < chunk_off[lo + 1]
        while (hi - lo > 1) {
          const uint32_t mid = (lo + hi) >> 1;
          if (__ldg(&S.cx.chunk_off[mid]) <= c) lo = mid;
          else hi = mid;
        }
        walk_chunk(wk, lo, (c - __ldg(&S.cx.chunk_off[lo])) * 32u);
        have = true;
      } else {
        chunks_left = false;
      }
    }
    if (!have) {  // ---- a node from the queue
      uint32_t ticket = 0;
      if (lane == 0) ticket = atomicAdd(&q[Q_HEAD], 1u);
      ticket = __shfl_sync(FULL, ticket, 0);
      uint32_t got = 0;  // 1: the entry is there, 2: all work is done, 3: gave up
      if (lane == 0) {
        for (uint32_t polls = 0;; ++polls) {
          if (ticket < S.cx.q_cap && ld_acquire(&S.cx.queue[ticket].w) == tag) {
            got = 1;
            break;
          }
          if (ld_acquire(&q[Q_OUT]) == 0u) {
            got = 2;
            break;
          }
          if (polls > limit || ((polls & 63u) == 63u && ld_acquire(&S.counters[CNT_BAR_ERR]))) {
            if (polls > limit) diag(S, DIAG_WAIT_QUEUE);
            got = 3;
            break;
          }
          __nanosleep(polls < 8u ? 100 : 500);  // many warps read the same counters: back off
        }
      }
      got = __shfl_sync(FULL, got, 0);
      if (got != 1) {
        abandoned = got == 3;
        break;
      }
      const uint4 e = __ldcg(S.cx.queue + ticket);
      if (lane == 0) {
        uint32_t* st = wk.stack();
        st[0] = e.x;
        st[1] = (e.y & 0xFFFFu) | (e.z << 16);
        st[2] = (e.y >> 16) == 0xFFFFu ? NOF : (e.y >> 16);
      }
      wk.held = 1;
      __syncwarp();
    }
    // ---- depth first through what this warp holds
    while (wk.held) {
      const uint32_t k = --wk.held;
      __syncwarp();
      const uint32_t* st = wk.stack();
      const uint32_t node = st[3u * k], cj_ = st[3u * k + 1u], fr_ = st[3u * k + 2u];
      __syncwarp();
      walk_expand(wk, cj_ >> 16, node, cj_ & 0xFFFFu, fr_);
      wk.share();
    }
    __syncwarp();
    if (lane == 0) {
      __threadfence();
      atomicSub(&q[Q_OUT], 1u);
    }
  }
  if (abandoned && lane == 0) atomicExch(&S.counters[CNT_BAR_ERR], 1u);
  if (wk.big_mode) hset_clear_all(sw.w.hset, sw.w.hset_mask);
  if (lane == 0) {
    if (sw.n_computed | sw.n_created) {
      stat_add(S, CNT_STAT_CTX_TRANS, sw.n_computed);
      stat_add(S, CNT_STAT_CTX_STATES, sw.n_created);
      stat_add64(S, CNT_STAT_STEP_CYCLES, sw.cycles);
    }
    if (wk.n_frontier) stat_add(S, CNT_STAT_FRONTIER, wk.n_frontier);
    if (wk.n_nodes) stat_add(S, CNT_STAT_TASKS, wk.n_nodes);
    if (wk.n_tasks) stat_add(S, CNT_STAT_SHARED_NODES, wk.n_tasks);
    if (wk.n_frames) stat_add(S, CNT_STAT_FRAMES, wk.n_frames);
  }
}

// ===================================================================================== launchers

cudaError_t configure_walk_kernels() {
  return cudaFuncSetAttribute((const void*)ctx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
}

void launch_fill(const GrammarDev& G, const StateDev& S, int sweep_grid, cudaStream_t st, cudaEvent_t before_sweep,
                 cudaEvent_t after_sweep) {
  launch_plan(G, S, st);
  if (before_sweep) cudaEventRecord(before_sweep, st);
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
  ctx_init_kernel<<<std::min<uint32_t>(S.B, 148u), 1024, 0, st>>>(G, S);
  ctx_kernel<<<(unsigned)sweep_grid, SWEEP_WARPS * 32, S.au.smem_bytes, st>>>(G, S);
  if (after_sweep) cudaEventRecord(after_sweep, st);
  launch_publish(S, st);
}

}  // namespace fmt
