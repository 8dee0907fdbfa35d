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
// One warp per job.  The last set of a pruned chart is sorted, origins ascending, and its own index
// is the largest origin there is, so the scanned / completed items (the set's kernel) come first
// and the predicted ones last.  The start chart's only kernel item is the augmented start item.

constexpr int ROOT_WARPS = 8;
constexpr uint32_t ROOT_ITEMS = 1024;  // items of a last set that can become a root (staged in shared memory)

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
    bool ok = R.on && n > 0 && n <= min(R.max_items, ROOT_ITEMS);
    if (ok) {
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
      ok = P >= 1 && P <= R.max_ph && nk >= 1;
      if (ok) {
        // ---- look the root up; add it if it is new (the protocol of the state cache: equal roots made
        // at the same moment meet in the same slot and the loser adopts the winner's)
        uint32_t slot = h & R.hash_mask;
        int32_t my_id = -1;
        uint32_t my_chart = 0;
        for (uint32_t probe = 0; probe < 256; ++probe) {
          uint32_t v = 0;
          if (lane == 0) v = ld_acquire(&R.hash[slot]);
          v = __shfl_sync(FULL, v, 0);
          if (v == 0) {
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
              if (id < 0) break;  // the directory is full: this row walks the whole trie itself
              uint32_t* c = R.charts + coff;  // a chart of P empty sets and the root set
              for (uint32_t i = lane; i < CH_HDR + P + 2; i += 32) {
                uint32_t v2 = 0u;
                if (i == CH_SETS) v2 = P + 1;
                else if (i == CH_ITEMS) v2 = n;
                else if (i == CH_WORDS) v2 = words;
                else if (i == CH_HDR + P + 1) v2 = n;
                c[i] = v2;
              }
              for (uint32_t i = lane; i < n; i += 32) c[CH_HDR + P + 2 + i] = stage[i];
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
            if (old == 0) {  // entered: this fill sweeps it
              root = (uint32_t)my_id;
              if (lane == 0) {
                const uint32_t rj = atomicAdd(&R.counters[CNT_N_JOBS], 1u);
                R.rj_chart[rj] = my_chart;
                R.rj_mask[rj] = my_id;
                R.rj_flags[rj] = 0u;
                R.rj_jobs[rj] = rj;
              }
              break;
            }
            v = old;
          }
          const uint32_t rid = v - 1u;
          if (rid >= R.max_roots) break;
          const uint32_t* info = R.info + (size_t)rid * RI_WORDS;
          bool same = __ldcg(info + RI_HASH) == h && __ldcg(info + RI_NK) == nk && __ldcg(info + RI_N) == n && __ldcg(info + RI_P) == P;
          if (same) {
            const uint32_t* c = R.charts + __ldcg(info + RI_CHART) + CH_HDR + P + 2;
            for (uint32_t i = lane; i < nk; i += 32)
              if (__ldcg(c + i) != stage[i]) same = false;
          }
          same = __all_sync(FULL, same);
          if (same) {
            root = rid;
            break;
          }
          slot = (slot + 1u) & R.hash_mask;
        }
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
  __shared__ uint32_t sh[4];
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
  if (threadIdx.x == 0) {
    uint32_t fo = 0, so = 0, io = 0, f = failed ? 1u : 0u;
    if (!f) {
      fo = atomicAdd(&R.tops[TOP_FRONTIER], fr_total);
      so = atomicAdd(&R.tops[TOP_STATES], nst);
      io = atomicAdd(&R.tops[TOP_ITEMS], it_total);
      if (fo > R.fr_cap || fr_total > R.fr_cap - fo || so > R.st_cap || nst > R.st_cap - so || io > R.it_cap || it_total > R.it_cap - io) f = 1u;
    }
    sh[0] = fo, sh[1] = so, sh[2] = io, sh[3] = f;
  }
  __syncthreads();
  const uint32_t fr_off = sh[0], st_off = sh[1], it_off = sh[2];
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
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    info[RI_FR_OFF] = fr_off;
    info[RI_FR_N] = failed ? 0u : fr_total;
    info[RI_ST_OFF] = st_off;
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
// an accepting chart; block 0 also lists the work: the frontier of every job in chunks of 32 entries.
// A job without a usable root starts at the trie's first level with the chart's own last set.

__global__ void __launch_bounds__(1024) ctx_init_kernel(GrammarDev G, StateDev S) {
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  const RootDev& R = S.rt;
  const uint32_t Wm = G.Wm;
  auto ready = [&](const CtxJob& cj) { return cj.root != ROOT_NONE && __ldcg(R.info + (size_t)cj.root * RI_WORDS + RI_STATUS) == ROOT_READY; };
  for (uint32_t j = blockIdx.x; j < n_jobs; j += gridDim.x) {
    const CtxJob cj = S.cx.jobs[j];
    const uint32_t* src = ready(cj) ? R.ci_rows + (size_t)cj.root * Wm : nullptr;
    uint32_t* dst = S.mask_rows + (size_t)cj.mrow * Wm;
    const bool acc = (cj.row_acc >> 31) != 0u && G.eos >= 0;
    for (uint32_t w = threadIdx.x; w < Wm; w += blockDim.x) {
      uint32_t v = src ? src[w] : 0u;
      if (acc && w == ((uint32_t)G.eos >> 5)) v |= 1u << ((uint32_t)G.eos & 31u);
      dst[w] = v;
    }
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
// Origin codes of the sets a job's walk makes (see RootDev): a set of the row's chart, a set made
// by this walk, or a set of the root's region.  Items read from a region set carry the root's
// anonymous origins: placeholders are replaced by the chart sets the row binds them to.
struct WalkView {
  const uint32_t* base_off;
  const uint32_t* base_items;
  const uint16_t* bind;   // [P]
  uint32_t P;
  const uint2* rstates;   // the region's sets (first item, count)
  const uint32_t* ritems;
  const uint32_t* lrecs;  // the sets this walk has made
  uint32_t rec_words;
  const uint32_t* litems;
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
      const uint2 e = __ldg(rstates + (o - RBASE));
      p = ritems + e.x;
      n = e.y;
    }
  }
  // an item read from set o, in the walk's own naming
  __device__ __forceinline__ uint32_t fix(uint32_t item, uint32_t o) const {
    if (o < LBASE) return item;
    uint32_t oo = item >> 16;
    if (o < RBASE) return (oo == ORIGIN_SELF) ? ((o << 16) | (item & 0xFFFFu)) : item;
    if (oo == ORIGIN_SELF) oo = o;
    else if (oo < P) oo = bind[oo];
    else if (oo == P) oo = RBASE;                // the root set is set 0 of its region
    else oo = RBASE + (oo - P - 1u);             // the root sweep named its k-th set P + 1 + k
    return (oo << 16) | (item & 0xFFFFu);
  }
  __device__ __forceinline__ void ctx_reset(const WarpCtx&) const {}
  __device__ __forceinline__ bool ctx_hit(const WarpCtx&) const { return false; }
};

constexpr uint32_t SPILL_WORDS = 3u * 4096u;                // room for 4096 spilled nodes (node, set, job)
constexpr uint32_t V_DEAD = 0xFFFFFFu, V_PEND = 0xFFFFFEu;  // values of a remembered transition (24 bits)
constexpr uint32_t PS_CHART = 0xFFFFu;                      // "parent set" of a job without a root: the chart's last set

struct Walker {
  const GrammarDev& G;
  const StateDev& S;
  SweepWarp& sw;
  uint32_t* big;
  bool big_mode = false;
  uint32_t n_frontier = 0, n_tasks = 0;
  // Nodes that found the queue full wait at the top of the warp's large scratch area (the sets under
  // construction use the part below) and are expanded by this warp itself, last in first out.
  uint32_t spill_n = 0;
  __device__ __forceinline__ uint32_t* spill() const { return big + (S.big_arena_items - SPILL_WORDS); }

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
  __device__ __forceinline__ WalkView view(const CtxJob& cj, const JobCtx& J, uint32_t j) const {
    WalkView v;
    v.base_off = J.base_off;
    v.base_items = J.base_items;
    v.bind = S.cx.bind + (size_t)j * S.rt.max_ph;
    v.P = cj.pad[0] ? cj.P : 0u;
    v.rstates = S.rt.states + cj.st_off;
    v.ritems = S.rt.items;
    v.lrecs = J.recs;
    v.rec_words = S.au.rec_words;
    v.litems = S.au.items;
    return v;
  }
  __device__ void break_row(const JobCtx& J) {
    if (lane_id() == 0) {
      if (!(atomicOr(&S.row_flags[J.row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
      atomicExch(&S.counters[CNT_ERR], 1u);
    }
  }
  // One Earley step of job j from the set with origin code `pcode` on `byte` (all lanes, uniform
  // arguments): the id of the set reached, or T_DEAD (also when a capacity ran out: the row is
  // marked broken then, its mask is not used).
  __device__ uint32_t step(const CtxJob& cj, uint32_t j, uint32_t pcode, uint32_t byte) {
    const JobCtx J = job(cj, j);
    const WalkView v = view(cj, J, j);
    const uint32_t* pitems;
    uint32_t plen;
    v(pcode, pitems, plen);
    uint32_t r = sw.step(J, v, pitems, plen, pcode, byte, !big_mode);
    if (r == T_FAIL && !big_mode) {  // a set outgrew the shared-memory scratch: use the large area from now on
      big_mode = true;
      hset_clear_all(sw.w.hset, sw.w.hset_mask);
      clear_nt(G, sw.w);
      sw.w.cur = big;
      sw.w.cur_cap = S.big_arena_items - SPILL_WORDS;
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
  // Queue the nodes of the lanes with `want` (each alive, in set `state`, with children) for expansion.
  __device__ void push(const CtxJob& cj, uint32_t j, bool want, uint32_t node, uint32_t state) {
    const uint32_t lane = lane_id();
    const uint32_t wb = __ballot_sync(FULL, want);
    if (!wb) return;
    const uint32_t n = __popc(wb);
    uint32_t base = 0;
    if (lane == 0) {
      base = atomicAdd(&S.cx.qctr[Q_TAIL], n);
      const uint32_t fit = base >= S.cx.q_cap ? 0u : min(n, S.cx.q_cap - base);
      atomicAdd(&S.cx.qctr[Q_OUT], fit);  // (before this warp reports its own unit done)
    }
    base = __shfl_sync(FULL, base, 0);
    const uint32_t at = base + __popc(wb & ((1u << lane) - 1u));
    bool lost = false;
    if (want) {
      if (at < S.cx.q_cap) {
        uint4* e = S.cx.queue + at;
        e->x = node, e->y = state, e->z = j;
        __threadfence();
        st_release32(&e->w, (S.gen_ctx << 16) | 1u);
      } else {
        lost = true;  // the queue is full: this warp keeps the node for itself
      }
    }
    n_tasks += n;
    const uint32_t lb = __ballot_sync(FULL, lost);
    if (lb) {
      const uint32_t room = SPILL_WORDS / 3u;
      const uint32_t k = spill_n + __popc(lb & ((1u << lane) - 1u));
      bool gone = false;
      if (lost) {
        uint32_t* sp = spill();
        if (k < room) sp[3u * k] = node, sp[3u * k + 1u] = state, sp[3u * k + 2u] = j;
        else gone = true;
      }
      spill_n = min(spill_n + __popc(lb), room);
      __syncwarp();
      if (lane == 0) diag(S, DIAG_QUEUE_FULL);
      if (__any_sync(FULL, gone)) break_row(job(cj, j));  // (not even the spill area could hold it)
    }
  }
};

__device__ void walk_expand(Walker& wk, uint32_t j, uint32_t node, uint32_t state);

// Expand the nodes this warp had to keep because the queue was full.
__device__ void walk_drain(Walker& wk) {
  while (wk.spill_n) {
    const uint32_t k = --wk.spill_n;
    __syncwarp();
    const uint32_t* sp = wk.spill();
    const uint32_t node = sp[3u * k], state = sp[3u * k + 1u], j = sp[3u * k + 2u];
    __syncwarp();
    walk_expand(wk, j, node, state);
  }
}

// A chunk of 32 frontier entries of job j, one per lane: the transition out of the entry's parent set
// is looked up in the job's table (computed by this warp if nobody has yet); nodes reached alive
// mark their tokens and are queued for expansion if they have children.
__device__ void walk_chunk(Walker& wk, uint32_t j, uint32_t e0) {
  const GrammarDev& G = wk.G;
  const StateDev& S = wk.S;
  const uint32_t lane = lane_id();
  const CtxJob cj = S.cx.jobs[j];
  const bool use_root = cj.pad[0] != 0u;
  const uint32_t e = e0 + lane;
  const bool valid = e < cj.fr_n;
  uint32_t node = 0, ps = PS_CHART, eq = 0;
  if (valid) {
    if (use_root) {
      const uint2 fe = __ldg(S.rt.frontier + cj.fr_off + e);
      node = fe.x, ps = fe.y & 0xFFFFu, eq = fe.y >> 16;
    } else {
      node = cj.fr_off + e;
      eq = G.eq_of_byte[__ldg(&G.node_byte[node])];
    }
  }
  const uint32_t byte = valid ? __ldg(&G.node_byte[node]) : 0u;
  const uint32_t key = (ps << 8) | eq;  // 24 bits
  const unsigned long long gen = S.gen_ctx & 0xFFFFu;
  unsigned long long* tab = S.cx.ctab + (size_t)j * CT_SLOTS;
  // ---- one lane per distinct key asks the table
  const uint32_t peers = __match_any_sync(FULL, valid ? key : (0xFF000000u | lane));  // (a key has 24 bits: idle lanes match nobody)
  const bool leader = valid && (uint32_t)(__ffs(peers) - 1) == lane;
  uint32_t val = V_PEND;
  int slot = -1;       // >= 0: the slot that holds (or will hold) the value
  bool mine = false;   // this lane computes the value
  if (leader) {
    uint32_t s = (mix32(key) & (CT_SLOTS - 1));
    for (uint32_t probe = 0; probe < 64; ++probe) {
      unsigned long long v = ld_acquire64(tab + s);
      if ((v >> 48) != gen) {  // left by an earlier fill: free
        const unsigned long long nv = (gen << 48) | ((unsigned long long)key << 24) | V_PEND;
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
      if (((v >> 24) & 0xFFFFFFu) == key) {
        slot = (int)s;
        val = (uint32_t)v & 0xFFFFFFu;
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
    const uint32_t sps = __shfl_sync(FULL, ps, src), sbyte = __shfl_sync(FULL, byte, src);
    const uint32_t pcode = (sps == PS_CHART) ? cj.m - 1u : RBASE + sps;
    const uint32_t r = wk.step(cj, j, pcode, sbyte);
    if ((int)lane == src) {
      val = (r == T_DEAD) ? V_DEAD : r;
      if (slot >= 0) st_release64(tab + slot, (gen << 48) | ((unsigned long long)key << 24) | val);
    }
  }
  // ---- a value somebody else is computing: wait for it (the other warp is at it, it waits for nothing)
  if (leader && val == V_PEND) {
    const uint32_t limit = ctx_poll_limit(S, 22);
    for (uint32_t spin = 0; spin < limit; ++spin) {
      const unsigned long long v = ld_acquire64(tab + slot);
      val = (uint32_t)v & 0xFFFFFFu;
      if (val != V_PEND) break;
      __nanosleep(100);
    }
    if (val == V_PEND) {
      diag(S, DIAG_WAIT_VALUE);
      atomicExch(&S.counters[CNT_BAR_ERR], 1u);
      val = V_DEAD;
    }
  }
  val = __shfl_sync(FULL, val, __ffs(peers) - 1);
  const bool alive = valid && val != V_DEAD;
  if (alive) wk.mark_tokens(cj, node);
  const bool kids = alive && __ldg(&G.child_off[node + 1]) > __ldg(&G.child_off[node]);
  wk.push(cj, j, kids, node, val);
  wk.n_frontier += __popc(__ballot_sync(FULL, valid));
}

// The children of `node`, reached in set `state` (one this walk made) by job j.
__device__ void walk_expand(Walker& wk, uint32_t j, uint32_t node, uint32_t state) {
  const GrammarDev& G = wk.G;
  const StateDev& S = wk.S;
  const AutoDev& A = S.au;
  const uint32_t lane = lane_id();
  const CtxJob cj = S.cx.jobs[j];
  uint32_t* rec = A.recs + ((size_t)j * A.cap + state) * A.rec_words;
  const uint32_t c0 = __ldg(&G.child_off[node]), c1 = __ldg(&G.child_off[node + 1]);
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
      const uint32_t r = wk.step(cj, j, LBASE + state, sbyte);
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
    wk.push(cj, j, kids, c, t);
  }
}

// The walk of all jobs of a fill.  Work units: first the chunks of frontier entries, handed out by
// a counter; then node expansions, drawn from a queue that the units themselves feed.  A warp that
// finds the queue empty waits for either a new entry or the count of unfinished units to reach zero.
// No unit ever waits for another unit, only for a single Earley step that another warp is computing,
// so every wait ends; all the same each is a poll with a limit that flags an error instead of hanging.
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
  bool abandoned = false;

  // ---- the frontier chunks
  for (;;) {
    uint32_t c = 0;
    if (lane == 0) c = atomicAdd(&q[Q_CHUNK], 1u);
    c = __shfl_sync(FULL, c, 0);
    if (c >= n_chunks) break;
    uint32_t lo = 0, hi = n_jobs;  // the job whose chunks include c: chunk_off[lo] <= c < chunk_off[lo + 1]
    while (hi - lo > 1) {
      const uint32_t mid = (lo + hi) >> 1;
      if (__ldg(&S.cx.chunk_off[mid]) <= c) lo = mid;
      else hi = mid;
    }
    walk_chunk(wk, lo, (c - __ldg(&S.cx.chunk_off[lo])) * 32u);
    walk_drain(wk);
    __syncwarp();
    if (lane == 0) {
      __threadfence();
      atomicSub(&q[Q_OUT], 1u);
    }
  }
  // ---- the queue
  const uint32_t tag = (S.gen_ctx << 16) | 1u;
  const uint32_t limit = ctx_poll_limit(S, 22);
  for (;;) {
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
    walk_expand(wk, e.z, e.x, e.y);
    walk_drain(wk);
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
    if (wk.n_tasks) stat_add(S, CNT_STAT_TASKS, wk.n_tasks);
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
