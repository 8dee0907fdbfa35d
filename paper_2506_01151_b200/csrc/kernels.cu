// CUDA kernels of the mask path (sm_100a): advance, plan / walk / publish of the mask fill, gather
// and the logits masking.  Integer work only: no tensor cores are involved anywhere.
#include <cuda_runtime.h>

#include <algorithm>

#include "../../include/fmt.h"
#include "chart_step.cuh"
#include "kernels.h"

namespace fmt {

// ===================================================================================== helpers

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint64_t ld_cg64(const uint64_t* p) {
  return (uint64_t)__ldcg(reinterpret_cast<const unsigned long long*>(p));
}
__device__ __forceinline__ void stat_add(const StateDev& S, uint32_t slot, uint32_t v) {
  atomicAdd(reinterpret_cast<unsigned long long*>(S.counters + slot), (unsigned long long)v);
}
__device__ __forceinline__ void stat_max(const StateDev& S, uint32_t slot, uint32_t v) { atomicMax(S.counters + slot, v); }

__device__ __forceinline__ uint32_t* private_buf(const StateDev& S, uint32_t row, uint32_t which) {
  return S.arena + ((size_t)row * 3u + which) * S.chart_words;
}

// Look the finished chart `ch` up in the state cache, inserting it if it is new and there is room.
// Returns (uniformly) the cache id and the word offset of the cached copy, or id -1 when the
// chart is not in the cache and could not be added.  Wait-free: concurrent inserts of equal
// charts meet in the same hash slot and the loser adopts the winner's entry.
__device__ int32_t intern_chart(const StateDev& S, const uint32_t* ch, uint64_t& off_out) {
  const uint32_t lane = lane_id();
  off_out = 0;
  if (!S.cache_on) return -1;
  const uint32_t words = ch[CH_WORDS];
  const uint32_t hlo = ch[CH_HASH_LO];
  uint32_t slot = hlo & S.ht_mask;
  int32_t my_id = -1;
  uint64_t my_off = 0;
  for (uint32_t probe = 0; probe < 512; ++probe) {
    uint32_t v = 0;
    if (lane == 0) v = ld_acquire(&S.ht[slot]);
    v = __shfl_sync(FULL, v, 0);
    if (v == 0) {
      if (my_id < 0) {
        unsigned long long off = 0;
        int32_t id = -1;
        if (lane == 0) {
          if (ld_acquire(&S.counters[CNT_N_STATES]) < S.max_states) {
            uint32_t got = atomicAdd(&S.counters[CNT_N_STATES], 1u);
            if (got < S.max_states) {
              unsigned long long need = (words + 31u) & ~31u;
              off = atomicAdd(reinterpret_cast<unsigned long long*>(S.counters + CNT_POOL_LO), need);
              if (off + need <= S.pool_words) id = (int32_t)got;
            }
          }
        }
        id = __shfl_sync(FULL, id, 0);
        off = __shfl_sync(FULL, off, 0);
        if (id < 0) return -1;  // the cache is full
        uint32_t* dst = S.arena + S.pool_base + off;
        for (uint32_t i = lane; i < words; i += 32) dst[i] = ch[i];
        if (lane == 0) {
          S.st_off[id] = S.pool_base + off;
          S.st_mask[id] = -1;
        }
        __syncwarp();
        __threadfence();
        my_id = id;
        my_off = S.pool_base + off;
      }
      uint32_t old = 0;
      if (lane == 0) old = atomicCAS(&S.ht[slot], 0u, (uint32_t)my_id + 1u);
      old = __shfl_sync(FULL, old, 0);
      if (old == 0) {
        off_out = my_off;
        return my_id;
      }
      v = old;  // somebody else took the slot meanwhile: compare with theirs
    }
    const uint32_t sid = v - 1u;
    if (sid >= S.max_states) return -1;
    const uint64_t poff = ld_cg64(&S.st_off[sid]);
    const uint32_t* other = S.arena + poff;
    bool same = (__ldcg(other + CH_WORDS) == words) && (__ldcg(other + CH_HASH_LO) == hlo);
    if (same)
      for (uint32_t i = lane; i < words; i += 32)
        if (__ldcg(other + i) != ch[i]) same = false;
    same = __all_sync(FULL, same);
    if (same) {
      off_out = poff;
      return (int32_t)sid;
    }
    slot = (slot + 1u) & S.ht_mask;
  }
  return -1;
}

// ===================================================================================== start chart

__global__ void __launch_bounds__(32) init_kernel(GrammarDev G, StateDev S, int32_t* result) {
  extern __shared__ uint32_t smem[];
  AdvScratch s = adv_scratch(smem);
  hset_clear_all(s.w.hset, s.w.hset_mask);
  uint32_t* dst = S.arena + S.init_off;
  int r = chart_init(G, s, dst, S.chart_words);
  if (lane_id() == 0) *result = r;
}

// one warp: put the start chart into the cache and record its id
__global__ void __launch_bounds__(32) intern_init_kernel(StateDev S, int32_t* init_state) {
  uint64_t off;
  int32_t id = intern_chart(S, S.arena + S.init_off, off);
  if (lane_id() == 0) *init_state = id;
}

// rows[i] (or rows 0..n-1) go back to the start chart
__global__ void reset_kernel(StateDev S, const uint32_t* rows, uint32_t n, const int32_t* init_state) {
  uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t row = rows ? rows[i] : i;
  if (row >= S.B) return;
  S.row_chart[row] = S.init_off;
  S.row_buf[row] = 255;
  S.row_state[row] = *init_state;
  S.row_flags[row] = 0;
  S.row_mask[row] = MASK_ZERO;
}

// ===================================================================================== advance

constexpr int ADV_WARPS = 4;

__global__ void __launch_bounds__(ADV_WARPS * 32) advance_kernel(GrammarDev G, StateDev S, const int32_t* tokens,
                                                                  int32_t* status) {
  extern __shared__ uint32_t smem[];
  const uint32_t warp = threadIdx.x >> 5, lane = lane_id();
  const uint32_t row = blockIdx.x * ADV_WARPS + warp;
  if (row >= S.B) return;
  AdvScratch s = adv_scratch(smem + (size_t)warp * ADV_WARP_WORDS);
  auto finish = [&](int32_t st) {
    if (status && lane == 0) status[row] = st;
  };
  const int32_t tok = tokens[row];
  if (tok == -1) return finish(FMT_OK);
  const uint32_t flags = S.row_flags[row];
  if (flags & ROW_FINISHED) return finish(FMT_ERR_FINISHED);
  if (tok < 0 || (uint32_t)tok >= G.V) return finish(FMT_ERR_INVALID_ARG);
  if (flags & ROW_BROKEN) return finish(FMT_ERR_CAPACITY);
  const uint32_t* cur = S.arena + S.row_chart[row];
  const uint32_t b0 = __ldg(&G.vocab_off[tok]), b1 = __ldg(&G.vocab_off[tok + 1]);
  if (tok == G.eos) {
    if (cur[CH_FLAGS] & CHART_ACCEPTING) {
      if (lane == 0) S.row_flags[row] = flags | ROW_FINISHED;
      return finish(FMT_OK);
    }
    return finish(FMT_ERR_TOKEN_REJECTED);
  }
  if (b1 == b0) return finish(FMT_ERR_TOKEN_REJECTED);

  hset_clear_all(s.w.hset, s.w.hset_mask);
  for (uint32_t i = lane; i < ADV_NT_WORDS; i += 32) s.w.nt[i] = 0u;
  __syncwarp();
  // two private buffers that do not hold the current chart
  const uint32_t held = S.row_buf[row];
  const uint32_t t0 = (held == 0) ? 1u : 0u;
  const uint32_t t1 = (held == 2 || held == 255) ? (t0 == 0 ? 1u : 2u) : 2u;
  uint32_t which = t0;
  const uint32_t* src = cur;
  uint32_t* dst = nullptr;
  for (uint32_t i = b0; i < b1; ++i) {
    dst = private_buf(S, row, which);
    int r = chart_step(G, s, src, __ldg(&G.vocab_bytes[i]), dst, S.chart_words);
    if (r == 0) return finish(FMT_ERR_TOKEN_REJECTED);
    if (r < 0) {
      if (lane == 0) {
        S.row_flags[row] = flags | ROW_BROKEN;
        atomicExch(&S.counters[CNT_ERR], 1u);
        stat_add(S, CNT_STAT_CAPERR, 1u);
      }
      return finish(FMT_ERR_CAPACITY);
    }
    src = dst;
    which = (which == t0) ? t1 : t0;
    __syncwarp();
  }
  const uint32_t final_buf = (which == t0) ? t1 : t0;
  if (lane == 0) {
    stat_add(S, CNT_STAT_ADV, 1u);
    stat_max(S, CNT_STAT_ITEMS_MAX, dst[CH_ITEMS]);
    stat_max(S, CNT_STAT_SETS_MAX, dst[CH_SETS]);
  }
  uint64_t off;
  int32_t id = intern_chart(S, dst, off);
  if (lane == 0) {
    S.row_state[row] = id;
    if (id >= 0) {
      S.row_chart[row] = off;
      S.row_buf[row] = 255;
    } else {
      S.row_chart[row] = (uint64_t)(dst - S.arena);
      S.row_buf[row] = (uint8_t)final_buf;
    }
  }
  finish(FMT_OK);
}

// ===================================================================================== fill: plan

// One thread per row decides where the row's mask comes from.
__global__ void plan_kernel(GrammarDev G, StateDev S) {
  if (blockIdx.x == 0 && threadIdx.x == 0) S.counters[CNT_WORK] = 0u;
  const uint32_t row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= S.B) return;
  stat_add(S, CNT_STAT_FILLS, 1u);
  const uint32_t flags = S.row_flags[row];
  if (flags & ROW_BROKEN) {
    S.row_mask[row] = MASK_ZERO;
    return;
  }
  if (flags & ROW_FINISHED) {
    S.row_mask[row] = MASK_EOS_ONLY;
    return;
  }
  const int32_t sid = S.row_state[row];
  if (sid >= 0) {
    int32_t old = atomicCAS(&S.st_mask[sid], -1, -2 - (int32_t)row);
    if (old >= 0) {  // cached
      S.row_mask[row] = old;
      stat_add(S, CNT_STAT_CACHED, 1u);
      return;
    }
    if (old <= -2) {  // another row of this call computes it
      S.row_mask[row] = MASK_ALIAS0 - (-2 - old);
      stat_add(S, CNT_STAT_SHARED, 1u);
      return;
    }
    // this row computes it, into a cache row if one is left
    int32_t mrow = (int32_t)row;
    if (ld_acquire(&S.counters[CNT_N_MASK_ROWS]) < S.max_mask_rows) {
      uint32_t got = atomicAdd(&S.counters[CNT_N_MASK_ROWS], 1u);
      if (got < S.max_mask_rows) mrow = (int32_t)(S.B + got);
    }
    S.row_mask[row] = mrow;
  } else {
    S.row_mask[row] = (int32_t)row;
  }
  stat_add(S, CNT_STAT_COMPUTED, 1u);
  uint32_t j = atomicAdd(&S.counters[CNT_N_JOBS], 1u);
  S.jobs[j] = row;
}

// Zero the mask rows about to be computed and set their EOS bit.
__global__ void prepare_rows_kernel(GrammarDev G, StateDev S) {
  const uint32_t j = blockIdx.x;
  if (j >= S.counters[CNT_N_JOBS]) return;
  const uint32_t row = S.jobs[j];
  uint32_t* m = S.mask_rows + (size_t)S.row_mask[row] * G.Wm;
  for (uint32_t i = threadIdx.x; i < G.Wm; i += blockDim.x) m[i] = 0u;
  __syncthreads();
  if (threadIdx.x == 0 && G.eos >= 0) {
    const uint32_t* ch = S.arena + S.row_chart[row];
    if (ch[CH_FLAGS] & CHART_ACCEPTING) m[(uint32_t)G.eos >> 5] |= 1u << ((uint32_t)G.eos & 31u);
  }
}

// ===================================================================================== fill: walk

constexpr int WALK_WARPS = 8;
constexpr uint32_t WALK_STAGE_WORDS = 4096;  // a base chart up to this size is staged in shared memory
constexpr uint32_t WALK_ARENA = 1024;        // items of level sets per warp (fast mode)
constexpr uint32_t WALK_HSET = 512;
constexpr uint32_t WALK_NT_WORDS = 256;      // 2 * Nw
constexpr uint32_t WALK_LEVELS = MAX_TOKEN_BYTES + 1;
constexpr uint32_t UNITS_PER_CHUNK = 64;

struct Frame {
  uint32_t node, cursor, pending, batch, set_off, set_len;
  uint32_t scan[8];
};
constexpr uint32_t FRAME_WORDS = sizeof(Frame) / 4;
constexpr uint32_t WALK_PATH_WORDS = (MAX_TOKEN_BYTES + 4) / 4 + 1;
constexpr uint32_t WALK_WARP_WORDS =
    WALK_ARENA + WALK_HSET + WALK_LEVELS * FRAME_WORDS + WALK_NT_WORDS + W_CTRS + WALK_PATH_WORDS;
constexpr uint32_t WALK_BLOCK_WORDS = WALK_STAGE_WORDS + 16;

struct Walker {
  const GrammarDev& G;
  WarpCtx w;
  uint32_t* arena;
  uint32_t arena_cap;
  Frame* frames;
  uint8_t* path;
  const uint32_t* base_off;
  const uint32_t* base_items;
  uint32_t m;  // live sets of the base chart
  uint32_t* mask_row;
  uint32_t top;  // items in use in the arena

  struct View {
    const Walker& wk;
    __device__ __forceinline__ void operator()(uint32_t o, const uint32_t*& p, uint32_t& n) const {
      if (o < wk.m) {
        uint32_t a = wk.base_off[o], b = wk.base_off[o + 1];
        p = wk.base_items + a;
        n = b - a;
      } else {
        const Frame& f = wk.frames[o - (wk.m - 1)];
        p = wk.arena + f.set_off;
        n = f.set_len;
      }
    }
  };

  __device__ __forceinline__ void emit_tokens(uint32_t node) const {
    uint32_t a = __ldg(&G.tok_off[node]), b = __ldg(&G.tok_off[node + 1]);
    for (uint32_t i = a; i < b; ++i) {
      uint32_t t = __ldg(&G.tok_ids[i]);
      atomicOr(&mask_row[t >> 5], 1u << (t & 31u));
    }
  }

  // The Earley set of trie depth `level`, reached from `parent` by `byte`:
  // scan, complete, predict; no pruning inside a token.  1 ok, 0 empty, -1 overflow.
  __device__ int step(const uint32_t* parent, uint32_t plen, uint32_t level, uint32_t byte) {
    const uint32_t lane = lane_id();
    if (top + 64 > arena_cap) return -1;
    w.cur = arena + top;
    w.cur_cap = arena_cap - top;
    __syncwarp();
    if (lane < W_CTRS) w.ctr[lane] = 0u;
    __syncwarp();
    uint32_t n = scan_into_cur(G, w, parent, plen, byte);
    if (w.ctr[W_OVERFLOW]) {
      hset_clear_all(w.hset, w.hset_mask);
      return -1;
    }
    if (n == 0) return 0;
    const uint32_t cur_index = m - 1 + level;
    complete_fixpoint(G, w, View{*this}, cur_index, 0u);
    uint32_t hashed = min(w.ctr[W_NCUR], w.cur_cap);
    if (w.ctr[W_OVERFLOW]) {
      hset_clear_all(w.hset, w.hset_mask);
      clear_nt(G, w);
      return -1;
    }
    hset_clear_items(w, hashed);
    predict_into_cur(G, w, cur_index);
    if (w.ctr[W_OVERFLOW]) return -1;
    n = drop_completed(G, w, min(w.ctr[W_NCUR], w.cur_cap));
    if (lane == 0) {
      frames[level].set_off = top;
      frames[level].set_len = n;
    }
    __syncwarp();
    top += n;
    return 1;
  }

  __device__ __forceinline__ void open_frame(uint32_t level, uint32_t node) {
    Frame& f = frames[level];
    __syncwarp();
    if (lane_id() == 0) {
      f.node = node;
      f.cursor = __ldg(&G.child_off[node]);
      f.pending = 0;
      f.batch = 0;
    }
    __syncwarp();
    scannable_bytes(G, arena + f.set_off, f.set_len, f.scan);
  }

  // One work unit.  1 done, -1 overflow.
  __device__ int unit(uint32_t u, const uint32_t* base_scan) {
    const uint32_t lane = lane_id();
    const uint32_t root = __ldg(&G.unit_node[u]);
    const uint32_t kind = __ldg(&G.unit_kind[u]);
    const uint32_t dr = __ldg(&G.node_depth[root]);
    if (dr == 0 || dr >= WALK_LEVELS) return 1;
    __syncwarp();
    if (lane == 0) {
      uint32_t n = root;
      for (uint32_t i = dr; i >= 1; --i) {
        path[i] = __ldg(&G.node_byte[n]);
        n = __ldg(&G.parent[n]);
      }
    }
    __syncwarp();
    const uint32_t first = path[1];
    if (!((base_scan[first >> 5] >> (first & 31u)) & 1u)) return 1;  // the first byte cannot follow
    top = 0;
    const uint32_t* pset = base_items + base_off[m - 1];
    uint32_t plen = base_off[m] - base_off[m - 1];
    const uint32_t full_levels = kind ? dr - 1 : dr;
    for (uint32_t L = 1; L <= full_levels; ++L) {
      int r = step(pset, plen, L, path[L]);
      if (r <= 0) return r == 0 ? 1 : -1;
      pset = arena + frames[L].set_off;
      plen = frames[L].set_len;
    }
    if (kind) {  // the node alone: does its last byte scan?
      bool hit = false;
      const uint32_t byte = path[dr];
      for (uint32_t k = lane; k < plen; k += 32) {
        uint32_t inf = __ldg(&G.info[pset[k] & 0xFFFFu]);
        if ((inf >> INFO_KIND_SHIFT) == KIND_TERM && class_has(G, inf & INFO_ARG_MASK, byte)) hit = true;
      }
      if (__any_sync(FULL, hit) && lane == 0) emit_tokens(root);
      return 1;
    }
    if (lane == 0) emit_tokens(root);
    if (__ldg(&G.child_off[root + 1]) == __ldg(&G.child_off[root])) return 1;
    open_frame(dr, root);
    uint32_t depth = dr;
    for (;;) {
      Frame& f = frames[depth];
      __syncwarp();
      const uint32_t pending = f.pending;
      if (pending == 0) {
        const uint32_t c0 = f.cursor, cend = __ldg(&G.child_off[f.node + 1]);
        if (c0 >= cend) {
          top = f.set_off;
          if (depth == dr) break;
          --depth;
          continue;
        }
        const uint32_t c = c0 + lane;
        bool internal = false;
        if (c < cend) {
          const uint32_t b = __ldg(&G.node_byte[c]);
          if ((f.scan[b >> 5] >> (b & 31u)) & 1u) {
            emit_tokens(c);
            internal = __ldg(&G.child_off[c + 1]) > __ldg(&G.child_off[c]);
          }
        }
        const uint32_t bal = __ballot_sync(FULL, internal);
        __syncwarp();
        if (lane == 0) {
          f.pending = bal;
          f.batch = c0;
          f.cursor = c0 + 32;
        }
      } else {
        const uint32_t k = (uint32_t)__ffs(pending) - 1u;
        const uint32_t c = f.batch + k;
        const uint32_t poff = f.set_off, plen2 = f.set_len;
        __syncwarp();
        if (lane == 0) f.pending = pending & (pending - 1u);
        __syncwarp();
        if (depth + 1 >= WALK_LEVELS) continue;  // cannot happen: tokens are at most MAX_TOKEN_BYTES long
        int r = step(arena + poff, plen2, depth + 1, __ldg(&G.node_byte[c]));
        if (r < 0) return -1;
        if (r > 0) {
          ++depth;
          open_frame(depth, c);
        }
      }
    }
    return 1;
  }
};

__global__ void __launch_bounds__(WALK_WARPS * 32) walk_kernel(GrammarDev G, StateDev S) {
  extern __shared__ uint32_t smem[];
  uint32_t* stage = smem;
  uint32_t* base_scan = smem + WALK_STAGE_WORDS;  // [8]
  uint32_t* blk = smem + WALK_STAGE_WORDS + 8;     // [8]
  const uint32_t warp = threadIdx.x >> 5, lane = lane_id();
  uint32_t* mine = smem + WALK_BLOCK_WORDS + (size_t)warp * WALK_WARP_WORDS;
  uint32_t* sm_arena = mine;
  uint32_t* sm_hset = sm_arena + WALK_ARENA;
  Frame* frames = reinterpret_cast<Frame*>(sm_hset + WALK_HSET);
  uint32_t* nt = reinterpret_cast<uint32_t*>(frames) + WALK_LEVELS * FRAME_WORDS;
  uint32_t* ctr = nt + WALK_NT_WORDS;
  uint8_t* path = reinterpret_cast<uint8_t*>(ctr + W_CTRS);
  // the large scratch area of this warp (global memory)
  uint32_t* big = S.big_scratch + ((size_t)blockIdx.x * WALK_WARPS + warp) * ((size_t)S.big_arena_items + S.big_hset_slots);

  hset_clear_all(sm_hset, WALK_HSET - 1);
  for (uint32_t i = lane; i < WALK_NT_WORDS; i += 32) nt[i] = 0u;
  __syncwarp();
  const uint32_t n_chunks = (G.U + UNITS_PER_CHUNK - 1) / UNITS_PER_CHUNK;
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  const uint32_t total = n_jobs * n_chunks;

  for (;;) {
    __syncthreads();
    if (threadIdx.x == 0) {
      blk[0] = atomicAdd(&S.counters[CNT_WORK], 1u);
      blk[1] = 0u;
    }
    __syncthreads();
    const uint32_t item = blk[0];
    if (item >= total) return;
    const uint32_t job = item / n_chunks, chunk = item % n_chunks;
    const uint32_t row = S.jobs[job];
    const uint32_t* chart = S.arena + S.row_chart[row];
    const uint32_t m = chart[CH_SETS], words = chart[CH_WORDS];
    const uint32_t* base = chart;
    if (words <= WALK_STAGE_WORDS) {
      for (uint32_t i = threadIdx.x; i < words; i += blockDim.x) stage[i] = chart[i];
      base = stage;
    }
    __syncthreads();
    const uint32_t* base_off = base + CH_HDR;
    const uint32_t* base_items = base + CH_HDR + m + 1;
    if (warp == 0) scannable_bytes(G, base_items + base_off[m - 1], base_off[m] - base_off[m - 1], base_scan);
    __syncthreads();

    Walker wk{G};
    wk.w.hset = sm_hset;
    wk.w.hset_mask = WALK_HSET - 1;
    wk.w.nt = nt;
    wk.w.ctr = ctr;
    wk.arena = sm_arena;
    wk.arena_cap = WALK_ARENA;
    wk.frames = frames;
    wk.path = path;
    wk.base_off = base_off;
    wk.base_items = base_items;
    wk.m = m;
    wk.mask_row = S.mask_rows + (size_t)S.row_mask[row] * G.Wm;
    wk.top = 0;
    bool big_mode = false;
    for (;;) {
      uint32_t k = 0;
      if (lane == 0) k = atomicAdd(&blk[1], 1u);
      k = __shfl_sync(FULL, k, 0);
      const uint32_t u = chunk + k * n_chunks;
      if (u >= G.U) break;
      int r = wk.unit(u, base_scan);
      if (r < 0 && !big_mode) {  // redo the unit, and do the rest of this chunk, with the large scratch area
        big_mode = true;
        hset_clear_all(wk.w.hset, wk.w.hset_mask);
        wk.arena = big;
        wk.arena_cap = S.big_arena_items;
        wk.w.hset = big + S.big_arena_items;
        wk.w.hset_mask = S.big_hset_slots - 1;
        clear_nt(G, wk.w);
        if (lane == 0) stat_add(S, CNT_STAT_BIG, 1u);
        r = wk.unit(u, base_scan);
      }
      if (r < 0) {  // even the large area is too small: the row's mask cannot be trusted
        hset_clear_all(wk.w.hset, wk.w.hset_mask);
        clear_nt(G, wk.w);
        if (lane == 0) {
          atomicOr(&S.row_flags[row], ROW_BROKEN);
          atomicExch(&S.counters[CNT_ERR], 1u);
          stat_add(S, CNT_STAT_CAPERR, 1u);
        }
        break;
      }
    }
  }
}

// ===================================================================================== fill: publish / gather / apply

__device__ __forceinline__ int32_t resolve_mask_row(const StateDev& S, uint32_t row) {
  int32_t r = S.row_mask[row];
  if (r <= MASK_ALIAS0) r = S.row_mask[(uint32_t)(MASK_ALIAS0 - r)];
  if (S.row_flags[row] & ROW_BROKEN) r = MASK_ZERO;
  return r;
}

// Publish the masks computed in this call to the cache (or release the claim when the row had
// no cache row, or broke).
__global__ void publish_kernel(StateDev S) {
  const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  if (j < n_jobs) {
    const uint32_t row = S.jobs[j];
    const int32_t sid = S.row_state[row];
    const bool broken = S.row_flags[row] & ROW_BROKEN;
    if (sid >= 0) {
      const int32_t mrow = S.row_mask[row];
      S.st_mask[sid] = (!broken && mrow >= (int32_t)S.B) ? mrow : -1;
    }
  }
}
__global__ void end_fill_kernel(StateDev S) { S.counters[CNT_N_JOBS] = 0u; }

// mask_out[row][w] for every row
__global__ void gather_kernel(GrammarDev G, StateDev S, uint32_t* out, size_t stride_words) {
  const uint32_t row = blockIdx.y;
  const int32_t r = resolve_mask_row(S, row);
  const uint32_t* src = (r >= 0) ? S.mask_rows + (size_t)r * G.Wm : nullptr;
  uint32_t* dst = out + (size_t)row * stride_words;
  for (size_t i = blockIdx.x * blockDim.x + threadIdx.x; i < stride_words; i += (size_t)gridDim.x * blockDim.x) {
    uint32_t v = 0;
    if (i < G.Wm) {
      if (src) v = src[i];
      else if (r == MASK_EOS_ONLY && G.eos >= 0 && i == ((uint32_t)G.eos >> 5)) v = 1u << ((uint32_t)G.eos & 31u);
    }
    dst[i] = v;
  }
}

// logits[t] = -inf where bit t is 0, for one row.  Each thread handles 8 consecutive tokens
// (16 bytes of bf16, 32 bytes of fp32) when the row is 16-byte aligned, else one token at a time.
// Groups whose 8 tokens are all valid are not touched; groups whose 8 tokens are all invalid are
// stored without being read.
template <typename T>
__device__ __forceinline__ void apply_row(const uint32_t* mask_row, int32_t special, int32_t eos, T* logits, uint32_t V,
                                          uint32_t* mask_out) {
  const uint32_t nthreads = gridDim.x * blockDim.x;
  const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x;
  const bool aligned = (reinterpret_cast<uintptr_t>(logits) & 15u) == 0;
  const uint32_t groups = (V + 7) / 8;
  const T neg = sizeof(T) == 2 ? (T)0xFF80u : (T)0xFF800000u;
  for (uint32_t g = tid; g < groups; g += nthreads) {
    const uint32_t t0 = g * 8;
    uint32_t word = 0;
    if (mask_row) word = __ldg(&mask_row[t0 >> 5]);
    else if (special == MASK_EOS_ONLY && eos >= 0 && (t0 >> 5) == ((uint32_t)eos >> 5)) word = 1u << ((uint32_t)eos & 31u);
    if (mask_out && (t0 & 31u) == 0) mask_out[t0 >> 5] = word;
    const uint32_t bits = (word >> (t0 & 31u)) & 0xFFu;
    if (bits == 0xFFu) continue;
    if (aligned && t0 + 8 <= V) {
      if (sizeof(T) == 2) {
        uint4* p = reinterpret_cast<uint4*>(logits + t0);
        uint4 v = (bits == 0) ? make_uint4(0, 0, 0, 0) : *p;
        uint32_t* e = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t lo = (bits >> (2 * i)) & 1u, hi = (bits >> (2 * i + 1)) & 1u;
          uint32_t x = e[i];
          if (!lo) x = (x & 0xFFFF0000u) | 0xFF80u;
          if (!hi) x = (x & 0x0000FFFFu) | 0xFF800000u;
          e[i] = x;
        }
        *p = v;
      } else {
        uint4* p = reinterpret_cast<uint4*>(logits + t0);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t hb = (bits >> (4 * h)) & 0xFu;
          if (hb == 0xFu) continue;
          uint4 v = (hb == 0) ? make_uint4(0, 0, 0, 0) : p[h];
          if (!(hb & 1u)) v.x = 0xFF800000u;
          if (!(hb & 2u)) v.y = 0xFF800000u;
          if (!(hb & 4u)) v.z = 0xFF800000u;
          if (!(hb & 8u)) v.w = 0xFF800000u;
          p[h] = v;
        }
      }
    } else {
      for (uint32_t i = 0; i < 8 && t0 + i < V; ++i)
        if (!((bits >> i) & 1u)) logits[t0 + i] = neg;
    }
  }
}

template <typename T>
__global__ void apply_kernel(const uint32_t* mask, size_t stride_words, T* logits, uint32_t V, size_t row_stride) {
  const uint32_t row = blockIdx.y;
  apply_row<T>(mask + (size_t)row * stride_words, 0, -1, logits + (size_t)row * row_stride, V, nullptr);
}

template <typename T>
__global__ void gather_apply_kernel(GrammarDev G, StateDev S, T* logits, size_t row_stride, uint32_t* mask_out,
                                    size_t stride_words) {
  const uint32_t row = blockIdx.y;
  const int32_t r = resolve_mask_row(S, row);
  const uint32_t* src = (r >= 0) ? S.mask_rows + (size_t)r * G.Wm : nullptr;
  uint32_t* mo = mask_out ? mask_out + (size_t)row * stride_words : nullptr;
  apply_row<T>(src, r, G.eos, logits + (size_t)row * row_stride, G.V, mo);
  if (mo)  // padding words beyond ceil(V/32)
    for (size_t i = G.Wm + blockIdx.x * blockDim.x + threadIdx.x; i < stride_words; i += (size_t)gridDim.x * blockDim.x)
      mo[i] = 0u;
}

// ===================================================================================== cache clear, query

// Step 1 of a cache clear: rows whose chart lives in the pool copy it to private buffer 0.
__global__ void evacuate_kernel(StateDev S) {
  const uint32_t row = blockIdx.x;
  if (row >= S.B) return;
  const uint64_t off = S.row_chart[row];
  __syncthreads();
  if (off >= S.pool_base) {
    const uint32_t* src = S.arena + off;
    uint32_t* dst = private_buf(S, row, 0);
    const uint32_t words = src[CH_WORDS];
    for (uint32_t i = threadIdx.x; i < words; i += blockDim.x) dst[i] = src[i];
    __syncthreads();
    if (threadIdx.x == 0) {
      S.row_chart[row] = (uint64_t)(dst - S.arena);
      S.row_buf[row] = 0;
    }
  }
  if (threadIdx.x == 0) S.row_state[row] = -1;
}
// Step 3: the start chart (block B) and every row's chart go back into the now empty cache.
__global__ void __launch_bounds__(32) reintern_kernel(StateDev S, int32_t* init_state) {
  const uint32_t row = blockIdx.x;
  uint64_t off;
  if (row == S.B) {
    int32_t id = intern_chart(S, S.arena + S.init_off, off);
    if (lane_id() == 0) *init_state = id;
    return;
  }
  if (S.row_chart[row] == S.init_off) return;  // fixed up by the caller's second pass
  const uint32_t* ch = S.arena + S.row_chart[row];
  int32_t id = intern_chart(S, ch, off);
  if (lane_id() == 0 && id >= 0) {
    S.row_state[row] = id;
    S.row_chart[row] = off;
    S.row_buf[row] = 255;
  }
}
// Step 4: rows still at the start chart take the start chart's new id.
__global__ void fix_init_rows_kernel(StateDev S, const int32_t* init_state) {
  const uint32_t row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row < S.B && S.row_chart[row] == S.init_off) S.row_state[row] = *init_state;
}

__global__ void query_kernel(StateDev S, uint8_t* accepting, uint8_t* finished, uint32_t* n_sets, uint32_t* n_items,
                             int32_t* state_id) {
  const uint32_t row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= S.B) return;
  const uint32_t* ch = S.arena + S.row_chart[row];
  accepting[row] = (ch[CH_FLAGS] & CHART_ACCEPTING) ? 1 : 0;
  finished[row] = (S.row_flags[row] & ROW_FINISHED) ? 1 : ((S.row_flags[row] & ROW_BROKEN) ? 2 : 0);
  n_sets[row] = ch[CH_SETS];
  n_items[row] = ch[CH_ITEMS];
  state_id[row] = S.row_state[row];
}

// ===================================================================================== launchers

static inline cudaError_t opt_in_smem(const void* fn, size_t bytes) {
  return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

static size_t adv_smem_bytes() { return (size_t)ADV_WARPS * ADV_WARP_WORDS * 4; }
static size_t init_smem_bytes() { return (size_t)ADV_WARP_WORDS * 4; }
static size_t walk_smem_bytes() { return ((size_t)WALK_BLOCK_WORDS + (size_t)WALK_WARPS * WALK_WARP_WORDS) * 4; }
int walk_warps() { return WALK_WARPS; }

cudaError_t configure_kernels() {
  cudaError_t e;
  if ((e = opt_in_smem((const void*)init_kernel, init_smem_bytes())) != cudaSuccess) return e;
  if ((e = opt_in_smem((const void*)advance_kernel, adv_smem_bytes())) != cudaSuccess) return e;
  if ((e = opt_in_smem((const void*)walk_kernel, walk_smem_bytes())) != cudaSuccess) return e;
  return cudaSuccess;
}

cudaError_t walk_blocks_per_sm(int* out) {
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(out, walk_kernel, WALK_WARPS * 32, walk_smem_bytes());
}

void launch_init(const GrammarDev& G, const StateDev& S, int32_t* result_dev, cudaStream_t st) {
  init_kernel<<<1, 32, init_smem_bytes(), st>>>(G, S, result_dev);
}
void launch_intern_init(const StateDev& S, int32_t* init_state_dev, cudaStream_t st) {
  intern_init_kernel<<<1, 32, 0, st>>>(S, init_state_dev);
}
void launch_reset(const StateDev& S, const uint32_t* rows_dev, uint32_t n, const int32_t* init_state_dev, cudaStream_t st) {
  if (n == 0) return;
  reset_kernel<<<(n + 127) / 128, 128, 0, st>>>(S, rows_dev, n, init_state_dev);
}
void launch_advance(const GrammarDev& G, const StateDev& S, const int32_t* tokens, int32_t* status, cudaStream_t st) {
  advance_kernel<<<(S.B + ADV_WARPS - 1) / ADV_WARPS, ADV_WARPS * 32, adv_smem_bytes(), st>>>(G, S, tokens, status);
}
void launch_fill(const GrammarDev& G, const StateDev& S, int walk_grid, cudaStream_t st, cudaEvent_t before_walk,
                 cudaEvent_t after_walk) {
  plan_kernel<<<(S.B + 255) / 256, 256, 0, st>>>(G, S);
  prepare_rows_kernel<<<S.B, 256, 0, st>>>(G, S);
  if (before_walk) cudaEventRecord(before_walk, st);
  walk_kernel<<<walk_grid, WALK_WARPS * 32, walk_smem_bytes(), st>>>(G, S);
  if (after_walk) cudaEventRecord(after_walk, st);
  publish_kernel<<<(S.B + 255) / 256, 256, 0, st>>>(S);
}
void launch_walk(const GrammarDev& G, const StateDev& S, int grid, cudaStream_t st) {
  walk_kernel<<<grid, WALK_WARPS * 32, walk_smem_bytes(), st>>>(G, S);
}
void launch_end_fill(const StateDev& S, cudaStream_t st) { end_fill_kernel<<<1, 1, 0, st>>>(S); }
void launch_gather(const GrammarDev& G, const StateDev& S, uint32_t* out, size_t stride_words, cudaStream_t st) {
  dim3 grid((unsigned)std::min<size_t>((stride_words + 255) / 256, 64), S.B);
  gather_kernel<<<grid, 256, 0, st>>>(G, S, out, stride_words);
}
void launch_apply(const uint32_t* mask, size_t stride_words, void* logits, int dtype, uint32_t batch, uint32_t V,
                  size_t row_stride, cudaStream_t st) {
  if (batch == 0 || V == 0) return;
  dim3 grid((unsigned)std::min<uint32_t>(((V + 7) / 8 + 255) / 256, 64), batch);
  if (dtype == FMT_BF16) apply_kernel<uint16_t><<<grid, 256, 0, st>>>(mask, stride_words, (uint16_t*)logits, V, row_stride);
  else apply_kernel<uint32_t><<<grid, 256, 0, st>>>(mask, stride_words, (uint32_t*)logits, V, row_stride);
}
void launch_gather_apply(const GrammarDev& G, const StateDev& S, void* logits, int dtype, size_t row_stride,
                         uint32_t* mask_out, size_t stride_words, cudaStream_t st) {
  dim3 grid((unsigned)std::min<uint32_t>(((G.V + 7) / 8 + 255) / 256, 64), S.B);
  if (dtype == FMT_BF16)
    gather_apply_kernel<uint16_t><<<grid, 256, 0, st>>>(G, S, (uint16_t*)logits, row_stride, mask_out, stride_words);
  else
    gather_apply_kernel<uint32_t><<<grid, 256, 0, st>>>(G, S, (uint32_t*)logits, row_stride, mask_out, stride_words);
}
void launch_evacuate(const StateDev& S, cudaStream_t st) { evacuate_kernel<<<S.B, 128, 0, st>>>(S); }
void launch_reintern(const StateDev& S, int32_t* init_state_dev, cudaStream_t st) {
  reintern_kernel<<<S.B + 1, 32, 0, st>>>(S, init_state_dev);
  fix_init_rows_kernel<<<(S.B + 127) / 128, 128, 0, st>>>(S, init_state_dev);
}
void launch_query(const StateDev& S, uint8_t* a, uint8_t* f, uint32_t* ns, uint32_t* ni, int32_t* sid, cudaStream_t st) {
  query_kernel<<<(S.B + 127) / 128, 128, 0, st>>>(S, a, f, ns, ni, sid);
}

}  // namespace fmt
