// CUDA kernels of the mask path (sm_100a): advance, plan / sweep / publish of the mask fill, gather
// and the logits masking.  Integer work only: no tensor cores are involved anywhere.
#include <cuda_runtime.h>

#include <algorithm>

#include "../../include/fmt.h"
#include "chart_step.cuh"
#include "sweep_warp.cuh"
#include "kernels.h"

namespace fmt {

// ===================================================================================== helpers


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
        if (id < 0) {  // the cache is full: tell the host, which empties it before the next advance
          if (lane == 0 && S.full_flag) *reinterpret_cast<volatile uint32_t*>(S.full_flag) = 1u;
          return -1;
        }
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
      if (lane == 0 && S.st_ref) S.st_ref[sid] = 1;  // (found again)
      off_out = poff;
      return (int32_t)sid;
    }
    slot = (slot + 1u) & S.ht_mask;
  }
  return -1;
}

// ===================================================================================== transition cache
//
// What advancing the chart with cache id `sid` by `tok` leads to, if that is known: the next chart's
// cache id, TR_REJECT, or TR_UNSET (not known).  Called by one lane.
__device__ __forceinline__ uint32_t tr_slot(const StateDev& S, unsigned long long key) {
  return (mix32((uint32_t)key) ^ mix32((uint32_t)(key >> 32) * 0x9E3779B9u)) & S.tr_mask;
}
__device__ int32_t tr_lookup(const StateDev& S, int32_t sid, uint32_t tok) {
  const unsigned long long key = ((unsigned long long)((uint32_t)sid + 1u) << 32) | tok;
  uint32_t slot = tr_slot(S, key);
  for (uint32_t probe = 0; probe < 32; ++probe) {
    const unsigned long long k = __ldcg(S.tr_key + slot);
    if (k == 0ull) return TR_UNSET;
    if (k == key) {
      const int32_t v = (int32_t)ld_acquire(reinterpret_cast<const uint32_t*>(S.tr_val + slot));
      return (v >= 0 || v == TR_REJECT) ? v : TR_UNSET;
    }
    slot = (slot + 1u) & S.tr_mask;
  }
  return TR_UNSET;
}
// Remember the outcome (one lane).  The first to claim a slot for the key writes the value; a full
// neighbourhood simply leaves the pair unrecorded.
__device__ void tr_insert(const StateDev& S, int32_t sid, uint32_t tok, int32_t val) {
  const unsigned long long key = ((unsigned long long)((uint32_t)sid + 1u) << 32) | tok;
  uint32_t slot = tr_slot(S, key);
  for (uint32_t probe = 0; probe < 32; ++probe) {
    const unsigned long long k = atomicCAS(S.tr_key + slot, 0ull, key);
    if (k == 0ull) {
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(S.tr_val + slot), "r"(val) : "memory");
      return;
    }
    if (k == key) return;
    slot = (slot + 1u) & S.tr_mask;
  }
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


__global__ void __launch_bounds__(ADV_WARPS * 32, 1) advance_kernel(GrammarDev Gg, StateDev S, const int32_t* tokens,
                                                                  int32_t* status) {
  extern __shared__ __align__(16) uint32_t smem[];
  const uint32_t warp = threadIdx.x >> 5, lane = lane_id();
  const uint32_t row = blockIdx.x * ADV_WARPS + warp;
  GrammarDev G = Gg;
  if (Gg.hot_words * 4u <= HOT_TABLE_BYTES) {
    G = stage_hot_tables(Gg, smem + (size_t)ADV_WARPS * ADV_WARP_WORDS);
    __syncthreads();
  }
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
  // ---- has this chart been advanced by this token before?  (Section 5.2: the state cache)
  const int32_t sid = S.cache_on ? S.row_state[row] : -1;
  if (sid >= 0) {
    int32_t known = TR_UNSET;
    if (lane == 0) known = tr_lookup(S, sid, (uint32_t)tok);
    known = __shfl_sync(FULL, known, 0);
    if (known == TR_REJECT) return finish(FMT_ERR_TOKEN_REJECTED);
    if (known >= 0 && (uint32_t)known < S.max_states) {
      if (lane == 0) {
        S.row_state[row] = known;
        S.st_ref[known] = 1;
        S.row_chart[row] = ld_cg64(&S.st_off[known]);
        S.row_buf[row] = 255;
        stat_add(S, CNT_STAT_ADV, 1u);
        stat_add(S, CNT_STAT_ADV_HIT, 1u);
      }
      return finish(FMT_OK);
    }
  }

  hset_clear_all(s.w.hset, s.w.hset_mask);
  for (uint32_t i = lane; i < ADV_NT_WORDS; i += 32) s.w.nt[i] = 0u;
  __syncwarp();
  // a private buffer that does not hold the current chart
  const uint32_t held = S.row_buf[row];
  const uint32_t final_buf = (held == 0) ? 1u : 0u;
  uint32_t* dst = private_buf(S, row, final_buf);
  uint32_t* const sm_arena = s.w.cur;
  int r = token_step(G, s, cur, G.vocab_bytes + b0, b1 - b0, dst, S.chart_words, sm_arena, ADV_CUR_CAP);
  if (r == -2) {  // the token's sets outgrew shared memory: use the row's third private buffer as the arena
    uint32_t* big = private_buf(S, row, 2);
    uint32_t cap = 32;
    while (cap * 2u <= S.chart_words) cap *= 2u;
    hset_clear_all(s.w.hset, s.w.hset_mask);
    for (uint32_t i = lane; i < ADV_NT_WORDS; i += 32) s.w.nt[i] = 0u;
    __syncwarp();
    r = (held == 2) ? -1 : token_step(G, s, cur, G.vocab_bytes + b0, b1 - b0, dst, S.chart_words, big, cap);
  }
  if (r == 0) {
    if (sid >= 0 && lane == 0) tr_insert(S, sid, (uint32_t)tok, TR_REJECT);
    return finish(FMT_ERR_TOKEN_REJECTED);
  }
  if (r < 0) {
    if (lane == 0) {
      S.row_flags[row] = flags | ROW_BROKEN;
      atomicExch(&S.counters[CNT_ERR], 1u);
      stat_add(S, CNT_STAT_CAPERR, 1u);
    }
    return finish(FMT_ERR_CAPACITY);
  }
  if (lane == 0) {
    stat_add(S, CNT_STAT_ADV, 1u);
    stat_max(S, CNT_STAT_ITEMS_MAX, dst[CH_ITEMS]);
    stat_max(S, CNT_STAT_SETS_MAX, dst[CH_SETS]);
    stat_add(S, CNT_STAT_ADV_WORDS, cur[CH_WORDS] + dst[CH_WORDS]);
  }
  uint64_t off;
  int32_t id = intern_chart(S, dst, off);
  if (lane == 0) {
    if (sid >= 0 && id >= 0) tr_insert(S, sid, (uint32_t)tok, id);
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

// ===================================================================================== forced bytes
//
// Per row, the run of bytes that every continuation of the row's text must begin with (the keys and
// punctuation a JSON schema fixes, Section 5.1's JSON-Schema task): as long as the text is not a
// sentence and the last Earley set can scan exactly one byte, that byte is taken and the chart is
// stepped over it.  Nothing of the row changes: the sets made on the way live in the warp's scratch.
__global__ void __launch_bounds__(ADV_WARPS * 32, 1) forced_kernel(GrammarDev Gg, StateDev S, uint8_t* bytes_out,
                                                                   size_t stride, uint32_t* len_out, uint32_t max_len) {
  extern __shared__ __align__(16) uint32_t smem[];
  const uint32_t warp = threadIdx.x >> 5, lane = lane_id();
  const uint32_t row = blockIdx.x * ADV_WARPS + warp;
  GrammarDev G = Gg;
  if (Gg.hot_words * 4u <= HOT_TABLE_BYTES) {
    G = stage_hot_tables(Gg, smem + (size_t)ADV_WARPS * ADV_WARP_WORDS);
    __syncthreads();
  }
  if (row >= S.B) return;
  AdvScratch s = adv_scratch(smem + (size_t)warp * ADV_WARP_WORDS);
  int n = 0;
  if (!(S.row_flags[row] & (ROW_FINISHED | ROW_BROKEN)) && max_len > 0) {
    hset_clear_all(s.w.hset, s.w.hset_mask);
    for (uint32_t i = lane; i < ADV_NT_WORDS; i += 32) s.w.nt[i] = 0u;
    __syncwarp();
    const uint32_t* cur = S.arena + S.row_chart[row];
    n = token_step(G, s, cur, nullptr, min(max_len, MAX_TOKEN_BYTES), nullptr, 0u, s.w.cur, ADV_CUR_CAP,
                   bytes_out + (size_t)row * stride);
    if (n < 0) n = 0;
  }
  if (lane == 0) len_out[row] = (uint32_t)n;
}

// ===================================================================================== fill: plan

// One block decides, row by row, where each mask comes from: the state cache, another row of
// this call with the same chart, or a fresh computation (a "job").
__global__ void __launch_bounds__(1024) plan_kernel(GrammarDev G, StateDev S) {
  if (threadIdx.x < CNT_HASH_GEN - CNT_BAR) S.counters[CNT_BAR + threadIdx.x] = 0u;  // barrier and level counters
  if (threadIdx.x < CNT_LAST_LEVEL + 1 - CNT_LEVEL_TAKEN) S.counters[CNT_LEVEL_TAKEN + threadIdx.x] = 0u;
  if (threadIdx.x == 0) {
    S.counters[CNT_N_JOBS] = 0u;
    S.counters[CNT_N_FJOBS] = 0u;
    S.counters[CNT_AUTO_ITEMS] = 0u;
  }
  if (S.rt.counters) {  // the root sweep of this fill starts from clean counters, too
    if (threadIdx.x < CNT_HASH_GEN - CNT_BAR) S.rt.counters[CNT_BAR + threadIdx.x] = 0u;
    if (threadIdx.x < CNT_LAST_LEVEL + 1 - CNT_LEVEL_TAKEN) S.rt.counters[CNT_LEVEL_TAKEN + threadIdx.x] = 0u;
    if (threadIdx.x == 0) S.rt.counters[CNT_N_JOBS] = 0u, S.rt.counters[CNT_AUTO_ITEMS] = 0u;
  }
  __syncthreads();
  for (uint32_t row = threadIdx.x; row < S.B; row += blockDim.x) {
    stat_add(S, CNT_STAT_FILLS, 1u);
    const uint32_t flags = S.row_flags[row];
    if (flags & ROW_BROKEN) {
      S.row_mask[row] = MASK_ZERO;
      continue;
    }
    if (flags & ROW_FINISHED) {
      S.row_mask[row] = MASK_EOS_ONLY;
      continue;
    }
    const int32_t sid = S.row_state[row];
    if (sid >= 0) {
      int32_t old = atomicCAS(&S.st_mask[sid], -1, -2 - (int32_t)row);
      if (old >= 0) {  // cached
        S.st_ref[sid] = 1;  // (used again: it outlives the next emptying of the cache)
        S.row_mask[row] = old;
        stat_add(S, CNT_STAT_CACHED, 1u);
        continue;
      }
      if (old <= -2) {  // another row of this call computes it
        S.row_mask[row] = MASK_ALIAS0 - (-2 - old);
        stat_add(S, CNT_STAT_SHARED, 1u);
        continue;
      }
      // this row computes it, into a cache row if one is left
      int32_t mrow = (int32_t)row;
      if (ld_acquire(&S.counters[CNT_N_MASK_ROWS]) < S.max_mask_rows) {
        uint32_t got = atomicAdd(&S.counters[CNT_N_MASK_ROWS], 1u);
        if (got < S.max_mask_rows) mrow = (int32_t)(S.mrow_base + got);
      }
      if (mrow == (int32_t)row && S.full_flag) *reinterpret_cast<volatile uint32_t*>(S.full_flag) = 1u;  // no mask row left to cache it in
      S.row_mask[row] = mrow;
    } else {
      S.row_mask[row] = (int32_t)row;
    }
    stat_add(S, CNT_STAT_COMPUTED, 1u);
    uint32_t j = atomicAdd(&S.counters[CNT_N_JOBS], 1u);
    S.jobs[j] = row;
  }
}

// ===================================================================================== fill: sweep
//
// For every job (a row whose mask must be computed) and every trie node the sweep answers "is the
// Earley set reached by this node's bytes non-empty?".  Sets are hash-consed per job (AutoDev): a
// transition (set, byte class) is computed once, by whichever warp needs it first, with the
// warp-cooperative scan / complete / predict of earley_device.cuh; everybody else reads it from
// the set's record.  The trie is processed one depth at a time by the whole grid, one THREAD per
// (job, node): st[node] = transition(st[parent], byte).  Reads of parent, byte and writes of st
// are coalesced because nodes are numbered breadth first.  The depths are not separated by grid
// barriers: a CTA reports the end of its part of a depth's pass, its warps then serve the queued
// transitions (tickets) while the other CTAs finish, and go on to the next depth once all have
// reported; a node whose parent's transition is still being computed waits for that transition
// alone.  The kernel is launched cooperatively so that all CTAs are resident, and every wait is a
// poll with an iteration limit that flags an error instead of hanging.

// (phase 0 of the sweep) what later phases need to know about job j, in one 16-byte record
__device__ __forceinline__ void make_job_info(const StateDev& S, uint32_t j) {
  const uint32_t row = S.jobs[j];
  const uint64_t off = S.row_chart[row];
  const uint32_t* chart = S.arena + off;
  const uint32_t acc = (chart[CH_FLAGS] & CHART_ACCEPTING) ? 0x80000000u : 0u;
  S.au.job_info[j] = make_uint4((uint32_t)off, (uint32_t)(off >> 32), chart[CH_SETS], row | acc);
}

__device__ __forceinline__ JobCtx job_ctx(const StateDev& S, uint32_t j) {
  const AutoDev& A = S.au;
  const uint4 ji = __ldcg(A.job_info + j);
  JobCtx J;
  J.row = ji.w & 0x7FFFFFFFu;
  J.accepting = (ji.w >> 31) != 0u;
  const uint32_t* chart = S.arena + (((uint64_t)ji.y << 32) | ji.x);
  J.m = ji.z;
  J.base_off = chart + CH_HDR;
  J.base_items = chart + CH_HDR + J.m + 1;
  J.recs = A.recs + (size_t)j * A.cap * A.rec_words;
  J.hash = A.hash + (size_t)j * (A.hash_mask + 1);
  J.n_states = A.n_states + j;
  J.cap = min(A.cap, (ORIGIN_SELF - 1u > J.m) ? ORIGIN_SELF - 1u - J.m : 0u);
  if (S.ctx_mode) J.cap = min(J.cap, ORIGIN_SELF - 16u - RBASE);  // a root's sets are named RBASE + id later on
  J.st = A.st + (size_t)j * A.st_stride;
  return J;
}

// What the Earley set at `node` is, given that its mark says "pending": the transition it waited
// for has been computed meanwhile.  `parent_state` is the (final) state of its parent.
__device__ __forceinline__ uint32_t settled(const GrammarDev& G, const AutoDev& A, const JobCtx& J, uint32_t parent_state,
                                            uint32_t byte) {
  const uint32_t* slot = J.recs + (size_t)parent_state * A.rec_words + AR_TRANS + G.eq_of_byte[byte];
  return ld_acquire(slot);  // (the set it names was written before the transition was published)
}

constexpr uint32_t SWEEP_PER_LANE = 4;  // trie nodes per lane and pass iteration (independent loads in flight)

__global__ void __launch_bounds__(SWEEP_WARPS * 32, 1) sweep_kernel(GrammarDev Gg, StateDev S) {
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  if (n_jobs == 0) return;  // every CTA sees the same count: nobody is left at a barrier
  extern __shared__ __align__(16) uint32_t smem[];
  const uint32_t warp = threadIdx.x >> 5, lane = lane_id();
  const AutoDev& A = S.au;
  const uint32_t ntw = (2u * Gg.Nw + 7u) & ~7u;
  const uint32_t warp_words = SWEEP_CUR + SWEEP_HSET + ntw + W_CTRS + 8;
  uint32_t* mine = smem + (size_t)warp * warp_words;
  uint32_t* sm_cur = mine;
  uint32_t* sm_hset = sm_cur + SWEEP_CUR;
  uint32_t* nt = sm_hset + SWEEP_HSET;
  uint32_t* ctr = nt + ntw;
  uint32_t* tmp8 = ctr + W_CTRS;
  // ---- the small grammar tables every Earley step reads go to shared memory when they fit
  GrammarDev G = Gg;
  if (A.tables_in_smem) G = stage_hot_tables(Gg, smem + (size_t)SWEEP_WARPS * warp_words);
  uint32_t* big = S.big_scratch + ((size_t)blockIdx.x * SWEEP_WARPS + warp) * ((size_t)S.big_arena_items + S.big_hset_slots);
  const uint32_t gw = blockIdx.x * SWEEP_WARPS + warp, GW = gridDim.x * SWEEP_WARPS;
  uint32_t bar_phase = 0, pass_phase = 0;

  hset_clear_all(sm_hset, SWEEP_HSET - 1);
  for (uint32_t i = lane; i < ntw; i += 32) nt[i] = 0u;
  __syncthreads();

  // ---- the automata start with one state each: the base chart's last set
  for (uint32_t j = blockIdx.x; j < n_jobs; j += gridDim.x) {
    uint32_t* rec0 = A.recs + (size_t)j * A.cap * A.rec_words;
    for (uint32_t i = threadIdx.x; i < A.rec_words; i += blockDim.x)
      if (i < AR_SCAN || i >= AR_SCAN + 8) rec0[i] = (i >= AR_TRANS) ? T_UNKNOWN : 0u;
    if (threadIdx.x == 0) A.n_states[j] = 1u;
    if (warp == 0) {
      if (lane == 0) make_job_info(S, j);
      __syncwarp();
      __threadfence_block();
      JobCtx J = job_ctx(S, j);
      scannable_bytes(G, J.base_items + J.base_off[J.m - 1], J.base_off[J.m] - J.base_off[J.m - 1], tmp8);
      if (lane < 8) rec0[AR_SCAN + lane] = tmp8[lane];
    }
  }
  if (!grid_barrier(S, bar_phase)) return;

  SweepWarp sw{G, S};
  sw.gen = S.gen & 0xFFFFu;  // (a slot of the per-job hashes written under another generation counts as empty)
  sw.w.nt = nt;
  sw.w.ctr = ctr;
  sw.tmp8 = tmp8;
  sw.w.cur = sm_cur;
  sw.w.cur_cap = SWEEP_CUR;
  sw.w.hset = sm_hset;
  sw.w.hset_mask = SWEEP_HSET - 1;
  bool big_mode = false;

  uint32_t last_level = 0;
  uint32_t expect_req = n_jobs * Gg.n_eq;  // transitions likely to be queued at the next depth (depth 1: every byte class of every job)
  for (uint32_t L = 1; L <= G.depth; ++L) {
    const uint32_t lo = __ldg(&G.lvl_off[L]), hi = __ldg(&G.lvl_off[L + 1]);
    constexpr uint32_t CH = 32 * SWEEP_PER_LANE;
    const uint32_t nL = hi - lo, cpj = (nL + CH - 1) / CH;
    const uint32_t chunks = n_jobs * cpj;
    // ---- the pass: one thread per (job, node).  Known transitions are final; an unknown one is
    // claimed by the first thread that meets it, which queues it for the compute phase below, and
    // the node is marked pending.  A pending PARENT (marked at the previous depth, computed since)
    // is settled on the way; pending leaves are settled when the mask words are formed.
    bool any_alive = false;
    // a queued transition carries the fill's generation and the depth, so that whoever takes it can tell when it has landed
    const unsigned long long req_tag = ((unsigned long long)sw.gen << 48) | ((unsigned long long)L << 24);
    // the queue has two halves, used by odd and even depths in turn: a depth's transitions may still be
    // in the making while the next depth queues its own
    const uint32_t req_half = A.req_cap / 2u, req_base = (L & 1u) * req_half;
    for (uint32_t c = gw; c < chunks; c += GW) {
      const uint32_t j = c / cpj;
      const uint32_t first = lo + (c % cpj) * CH + lane;
      const JobCtx J = job_ctx(S, j);
      uint32_t node[SWEEP_PER_LANE], byte[SWEEP_PER_LANE], par[SWEEP_PER_LANE], ps[SWEEP_PER_LANE];
#pragma unroll
      for (uint32_t u = 0; u < SWEEP_PER_LANE; ++u) {
        node[u] = first + 32u * u;
        const bool v = node[u] < hi;
        byte[u] = v ? __ldg(&G.node_byte[node[u]]) : 0u;
        par[u] = (v && L > 1) ? __ldg(&G.parent[node[u]]) : 0u;
      }
#pragma unroll
      for (uint32_t u = 0; u < SWEEP_PER_LANE; ++u)
        ps[u] = (node[u] < hi) ? ((L == 1) ? 0u : (uint32_t)__ldcg(J.st + par[u])) : (uint32_t)ST_DEAD;  // written by other SMs: bypass L1
#pragma unroll
      for (uint32_t u = 0; u < SWEEP_PER_LANE; ++u) {
        if (node[u] >= hi) continue;
        uint32_t p_state = ps[u];
        if (p_state == ST_PENDING) {  // settle the parent first
          const uint32_t gp_state = (L == 2) ? 0u : (uint32_t)__ldcg(J.st + __ldg(&G.parent[par[u]]));
          uint32_t t2 = settled(G, A, J, gp_state, __ldg(&G.node_byte[par[u]]));
          // the transition was queued at the previous depth; the warp that drew it may still be at it
          for (uint32_t spin = 0; t2 == T_PENDING && spin < poll_limit(S, 21); ++spin) {
            __nanosleep(40);
            t2 = settled(G, A, J, gp_state, __ldg(&G.node_byte[par[u]]));
          }
          if (t2 == T_UNKNOWN || t2 == T_PENDING) {  // the wait ran out: give the row up rather than guess
            diag(S, DIAG_WAIT_VALUE);
            if (!(atomicOr(&S.row_flags[J.row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
            atomicExch(&S.counters[CNT_ERR], 1u);
            p_state = ST_DEAD;
          } else {
            p_state = (t2 == T_DEAD) ? (uint32_t)ST_DEAD : (t2 == T_CTX) ? (uint32_t)ST_CTX : t2;
          }
          J.st[par[u]] = (uint16_t)p_state;
        }
        uint32_t t = T_DEAD;
        if (p_state != ST_DEAD && p_state != ST_CTX) {  // (what lies below a context-dependent node is not this sweep's business)
          // records are written by other SMs while the sweep runs: read them past L1.  A record is complete
          // before its id appears anywhere (the writer fences, then publishes the transition that names it).
          const uint32_t* rec = J.recs + (size_t)p_state * A.rec_words;
          // one 256-bit test rejects most bytes without touching the transition table
          if ((__ldcg(rec + AR_SCAN + (byte[u] >> 5)) >> (byte[u] & 31u)) & 1u) {
            uint32_t* slot = J.recs + (size_t)p_state * A.rec_words + AR_TRANS + G.eq_of_byte[byte[u]];
            t = __ldcg(slot);  // (a final value is final; anything else is read again, in order)
            if (t == T_UNKNOWN || t == T_PENDING) t = ld_acquire(slot);
            if (t == T_UNKNOWN) {
              t = atomicCAS(slot, T_UNKNOWN, T_PENDING);
              if (t == T_UNKNOWN) {  // ours to queue
                const uint32_t at = atomicAdd(&S.counters[CNT_LEVEL_REQ + L], 1u);
                if (at < req_half) {
                  A.req[req_base + at] = req_tag | ((unsigned long long)j << 32) | ((unsigned long long)p_state << 8) | byte[u];
                  t = T_PENDING;
                } else {
                  // the depth's queue is full: nobody will compute this transition.  Settle it here so that
                  // nobody waits for it: the root sweep calls it context-dependent (always a safe answer),
                  // a row's own sweep gives the row up.
                  t = S.ctx_mode ? T_CTX : T_DEAD;
                  diag(S, DIAG_QUEUE_FULL);
                  if (!S.ctx_mode) {
                    if (!(atomicOr(&S.row_flags[J.row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
                    atomicExch(&S.counters[CNT_ERR], 1u);
                  }
                  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(slot), "r"(t) : "memory");
                }
              }
            }
          }
        }
        J.st[node[u]] = (t == T_PENDING) ? ST_PENDING : (t == T_DEAD) ? ST_DEAD : (t == T_CTX) ? ST_CTX : (uint16_t)t;
        any_alive |= (t != T_DEAD && t != T_CTX);
      }
    }
    __syncwarp();
    if (__any_sync(FULL, any_alive) && lane == 0) atomicOr(&S.counters[CNT_LEVEL_ALIVE + L], 1u);
    // ---- this CTA's part of the pass is done.  The queued transitions are computed WHILE the other
    // CTAs finish theirs: every warp draws a ticket and serves the transition with that number as
    // soon as it has been queued; a ticket beyond the last transition queued, once all CTAs are
    // done with the pass, is void.  One transition per warp at a time, all warps of the grid in parallel.
    if (!pass_arrive(S, pass_phase)) return;
    const uint32_t all_passed = pass_phase * gridDim.x;
    // When few transitions are being queued (as many as at the depth before, roughly), eight warps of
    // every CTA stand by for tickets and the others simply wait for them at the CTA's barrier below:
    // thousands of warps polling the same counters slow down the few that work.  A heavy fill
    // needs all hands.
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
        __nanosleep(polls < 16u ? 40 : 200);  // thousands of warps read the same two counters: back off
        continue;
      }
      polls = 0;
      unsigned long long rq = 0;
      if (lane == 0) {  // the entry is written right after its number was drawn: wait for it to land
        for (uint32_t spin = 0; spin < poll_limit(S, 22); ++spin) {
          rq = ld_acquire64(A.req + req_base + ticket);  // (a volatile access: a plain load may be hoisted out of the loop)
          if ((rq >> 48) == sw.gen && ((rq >> 24) & 0xFFu) == L) break;
          rq = 0;
        }
      }
      rq = __shfl_sync(FULL, rq, 0);
      have_ticket = false;
      if (rq == 0) {
        if (lane == 0) diag(S, DIAG_WAIT_QUEUE);
        gave_up = true;
        break;
      }
      const uint32_t j = (uint32_t)(rq >> 32) & 0xFFFFu, p_state = (uint32_t)(rq >> 8) & 0xFFFFu, pb = (uint32_t)rq & 0xFFu;
      const JobCtx J = job_ctx(S, j);
      uint32_t r = sw.compute(J, p_state, pb, !big_mode);
      if (r == T_FAIL && !big_mode) {  // a set outgrew the shared-memory scratch: use the large area from now on
        big_mode = true;
        hset_clear_all(sw.w.hset, sw.w.hset_mask);
        clear_nt(G, sw.w);
        sw.w.cur = big;
        sw.w.cur_cap = S.big_arena_items;
        sw.w.hset = big + S.big_arena_items;
        sw.w.hset_mask = S.big_hset_slots - 1;
        if (lane == 0) stat_add(S, CNT_STAT_BIG, 1u);
        r = sw.compute(J, p_state, pb, false);
      }
      if (r == T_FAIL) {  // a capacity was exceeded: the row's mask cannot be trusted
        hset_clear_all(sw.w.hset, sw.w.hset_mask);
        clear_nt(G, sw.w);
        if (lane == 0) {
          diag(S, DIAG_SET_SCRATCH);
          uint32_t* slot = J.recs + (size_t)p_state * A.rec_words + AR_TRANS + G.eq_of_byte[pb];
          if (S.ctx_mode) {  // the root sweep leaves what it cannot hold to the rows' own walks
            atomicExch(slot, T_CTX);
          } else {
            if (!(atomicOr(&S.row_flags[J.row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
            atomicExch(&S.counters[CNT_ERR], 1u);
            atomicExch(slot, T_DEAD);  // lets the sweep go on
          }
        }
      }
    }
    if (gave_up && lane == 0) atomicExch(&S.counters[CNT_BAR_ERR], 1u);  // cannot happen short of a fault elsewhere
    // all CTAs have passed this depth: how it went is read once per CTA, so that all its warps agree
    // (The next depth's pass starts at once: a node whose parent waits for a transition that is still
    // being computed waits for that one transition, see above.)
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
  // All CTAs have passed the last depth.  Transitions queued there may still be in the making: a
  // leaf that waits for one waits for it below, so no barrier is needed here either.
  {
    uint32_t abandoned = 0;
    if (lane == 0) abandoned = ld_acquire(&S.counters[CNT_BAR_ERR]);
    if (__shfl_sync(FULL, abandoned, 0) != 0u) return;  // the rows are marked broken when the masks are published
  }
  if (big_mode) hset_clear_all(sw.w.hset, sw.w.hset_mask);
  if (lane == 0 && (sw.n_computed | sw.n_created)) {
    stat_add(S, CNT_STAT_TRANS, sw.n_computed);
    stat_add(S, CNT_STAT_LOCAL, sw.n_created);
    stat_add64(S, CNT_STAT_STEP_CYCLES, sw.cycles);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) S.counters[CNT_LAST_LEVEL] = last_level;

  // ---- mask words: 32 tokens per warp pass, one ballot per word (token t is valid iff the node
  // where its bytes end was reached alive; EOS iff the chart is accepting)
  const uint32_t Wm = G.Wm;
  constexpr uint32_t MW = 6;  // mask words per warp and iteration: their loads are in flight together
  // nodes are numbered breadth first: a node was visited iff it comes before the first node of depth last_level + 1
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
      // where the word goes (needed last, asked for first: one lane, off the chain of the loads below)
      dst[u] = (valid[u] && lane == 0) ? (uint32_t)S.row_mask[__ldcg(A.job_info + c / Wm).w & 0x7FFFFFFFu] : 0u;
    }
#pragma unroll
    for (uint32_t u = 0; u < MW; ++u) {
      const uint32_t c = c0 + u * GW;
      s_[u] = ST_DEAD;
      eos_ok[u] = false;
      if (node[u] == 0xFFFFFFFFu) {  // a token without bytes: only EOS can be valid
        const uint32_t tok = (c % Wm) * 32 + lane;
        eos_ok[u] = ((int32_t)tok == G.eos) && !S.ctx_mode && job_ctx(S, c / Wm).accepting;
      } else if (node[u] < visited_end) {
        s_[u] = __ldcg(A.st + (size_t)(c / Wm) * A.st_stride + node[u]);
      }
    }
#pragma unroll
    for (uint32_t u = 0; u < MW; ++u) {
      if (!valid[u]) continue;  // (uniform)
      const uint32_t c = c0 + u * GW;
      const uint32_t j = c / Wm, wd = c % Wm;
      uint32_t s = s_[u];
      if (__any_sync(FULL, s == ST_PENDING)) {  // leaves that waited for a transition: their parents are final by now
        const JobCtx J = job_ctx(S, j);
        if (s == ST_PENDING) {
          const uint32_t p = __ldg(&G.parent[node[u]]);
          const uint32_t p_state = (p == 0) ? 0u : (uint32_t)__ldcg(J.st + p);
          uint32_t t2 = (p_state == ST_DEAD || p_state == ST_CTX || p_state == ST_PENDING) ? T_DEAD : settled(G, A, J, p_state, __ldg(&G.node_byte[node[u]]));
          for (uint32_t spin = 0; t2 == T_PENDING && spin < poll_limit(S, 21); ++spin) {  // some warp is still at it
            __nanosleep(40);
            t2 = settled(G, A, J, p_state, __ldg(&G.node_byte[node[u]]));
          }
          if (t2 == T_UNKNOWN || t2 == T_PENDING || p_state == ST_PENDING) {
            diag(S, DIAG_WAIT_VALUE);
            if (!(atomicOr(&S.row_flags[J.row], ROW_BROKEN) & ROW_BROKEN)) stat_add(S, CNT_STAT_CAPERR, 1u);
            s = ST_DEAD;
          } else {
            s = (t2 == T_DEAD) ? (uint32_t)ST_DEAD : (t2 == T_CTX) ? (uint32_t)ST_CTX : t2;
          }
          if (S.ctx_mode) J.st[node[u]] = (uint16_t)s;  // the frontier is collected from st afterwards
        }
      }
      const uint32_t word = __ballot_sync(FULL, (s != ST_DEAD && s != ST_CTX) || eos_ok[u]);
      if (lane == 0) S.mask_rows[(size_t)dst[u] * Wm + wd] = word;
    }
  }
}

// Publish the masks computed in this call to the cache (or release the claim when the row had
// no cache row, or broke).
__global__ void publish_kernel(StateDev S) {
  const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  if (j < n_jobs) {
    const uint32_t row = S.jobs[j];
    const int32_t sid = S.row_state[row];
    // a fill that was given up (a bounded wait ran out) hands out all-zero masks, never a guess; the
    // rows themselves are fine and the next fill computes them afresh
    const bool aborted = S.counters[CNT_BAR_ERR] != 0u;
    const bool broken = (S.row_flags[row] & ROW_BROKEN) || aborted;
    if (sid >= 0) {
      const int32_t mrow = S.row_mask[row];
      S.st_mask[sid] = (!broken && mrow >= (int32_t)S.B) ? mrow : -1;
    }
    if (aborted) {
      S.row_mask[row] = MASK_ZERO;
      if (j == 0) stat_add(S, CNT_STAT_ABORTS, 1u);
    }
  }
}

__device__ __forceinline__ int32_t resolve_mask_row(const StateDev& S, uint32_t row) {
  int32_t r = S.row_mask[row];
  if (S.row_flags[row] & ROW_BROKEN) return MASK_ZERO;
  if (r <= MASK_ALIAS0) {  // the mask another row of this call computed: not to be used if that row broke
    const uint32_t other = (uint32_t)(MASK_ALIAS0 - r);
    if (S.row_flags[other] & ROW_BROKEN) return MASK_ZERO;
    r = S.row_mask[other];
  }
  return r;
}

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

// logits[t] = -inf where bit t is 0, for one row, in groups of 8 tokens with 16-byte accesses when the
// row is 16-byte aligned, else token by token.  Groups whose 8 tokens are all
// valid are not touched; groups whose 8 tokens are all invalid are stored without being read.
template <typename T>
__device__ __forceinline__ void apply_group(T* p, uint32_t bits) {  // 8 tokens at p, 16-byte aligned
  if (sizeof(T) == 2) {
    uint4* q = reinterpret_cast<uint4*>(p);
    uint4 v = (bits == 0) ? make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u) : *q;
    if (bits != 0) {
      uint32_t* e = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t x = e[i];
        if (!((bits >> (2 * i)) & 1u)) x = (x & 0xFFFF0000u) | 0xFF80u;
        if (!((bits >> (2 * i + 1)) & 1u)) x = (x & 0x0000FFFFu) | 0xFF800000u;
        e[i] = x;
      }
    }
    *q = v;
  } else {
    uint4* q = reinterpret_cast<uint4*>(p);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t hb = (bits >> (4 * h)) & 0xFu;
      if (hb == 0xFu) continue;
      uint4 v = (hb == 0) ? make_uint4(0, 0, 0, 0) : q[h];
      if (!(hb & 1u)) v.x = 0xFF800000u;
      if (!(hb & 2u)) v.y = 0xFF800000u;
      if (!(hb & 4u)) v.z = 0xFF800000u;
      if (!(hb & 8u)) v.w = 0xFF800000u;
      q[h] = v;
    }
  }
}

template <typename T>
__device__ __forceinline__ void apply_row(const uint32_t* mask_row, int32_t special, int32_t eos, T* logits, uint32_t V,
                                          uint32_t* mask_out) {
  const uint32_t nthreads = gridDim.x * blockDim.x;
  const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x;
  const bool aligned = (reinterpret_cast<uintptr_t>(logits) & 15u) == 0;
  const uint32_t words = (V + 31) / 32;
  const T neg = sizeof(T) == 2 ? (T)0xFF80u : (T)0xFF800000u;
  auto word_at = [&](uint32_t wd) -> uint32_t {
    if (mask_row) return __ldg(&mask_row[wd]);
    return (special == MASK_EOS_ONLY && eos >= 0 && wd == ((uint32_t)eos >> 5)) ? 1u << ((uint32_t)eos & 31u) : 0u;
  };
  if (mask_out)
    for (uint32_t wd = tid; wd < words; wd += nthreads) mask_out[wd] = word_at(wd);
  if (aligned) {
    // consecutive lanes take consecutive groups of 8 tokens (16 bytes of bf16, 32 of fp32): every access of a
    // warp covers one contiguous piece of the row; four lanes share a mask word
    const uint32_t groups = V / 8;
#pragma unroll 4
    for (uint32_t gq = tid; gq < groups; gq += nthreads) {
      const uint32_t bits = (word_at(gq >> 2) >> (8u * (gq & 3u))) & 0xFFu;
      if (bits != 0xFFu) apply_group<T>(logits + (size_t)gq * 8, bits);
    }
    if (tid == 0)
      for (uint32_t t = groups * 8; t < V; ++t)
        if (!((word_at(t >> 5) >> (t & 31u)) & 1u)) logits[t] = neg;
  } else {
    for (uint32_t wd = tid; wd < words; wd += nthreads) {
      const uint32_t word = word_at(wd);
      if (word == 0xFFFFFFFFu) continue;
      const uint32_t t0 = wd * 32;
      for (uint32_t i = 0; i < 32 && t0 + i < V; ++i)
        if (!((word >> i) & 1u)) logits[t0 + i] = neg;
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
  if (off >= S.pool_lo) {
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

// Emptying the cache with survivors (see fmt_state_create's cache_keep_when_full): `Old` is the cache as it
// was - its charts, mask rows and tables are still intact in the other half of the storage -, S the emptied
// one.  Every entry of Old that was found again after it was made is entered into S, with its mask row.
__global__ void __launch_bounds__(32) survivors_kernel(GrammarDev G, StateDev Old, StateDev S, const uint32_t* old_count) {
  const uint32_t id = blockIdx.x * gridDim.y + blockIdx.y;
  if (id >= min(*old_count, Old.max_states) || !Old.st_ref[id]) return;
  const uint32_t lane = lane_id();
  uint64_t off;
  const int32_t nid = intern_chart(S, Old.arena + Old.st_off[id], off);
  if (nid < 0) return;  // no room: it goes after all
  const int32_t orow = Old.st_mask[id];
  if (orow < (int32_t)Old.B) return;  // no mask was kept for it
  uint32_t nrow = 0;
  if (lane == 0) {
    nrow = 0xFFFFFFFFu;
    if (S.st_mask[nid] == -1 && ld_acquire(&S.counters[CNT_N_MASK_ROWS]) < S.max_mask_rows) {
      const uint32_t got = atomicAdd(&S.counters[CNT_N_MASK_ROWS], 1u);
      if (got < S.max_mask_rows) nrow = S.mrow_base + got;
    }
  }
  nrow = __shfl_sync(FULL, nrow, 0);
  if (nrow == 0xFFFFFFFFu) return;
  const uint32_t* src = Old.mask_rows + (size_t)orow * G.Wm;
  uint32_t* dst = S.mask_rows + (size_t)nrow * G.Wm;
  for (uint32_t i = lane; i < G.Wm; i += 32) dst[i] = src[i];
  __syncwarp();
  if (lane == 0) S.st_mask[nid] = (int32_t)nrow;
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

static size_t adv_smem_bytes(const GrammarDev& G) {
  return (size_t)ADV_WARPS * ADV_WARP_WORDS * 4 + (G.hot_words * 4u <= HOT_TABLE_BYTES ? G.hot_words * 4u : 0u);
}
static size_t init_smem_bytes() { return (size_t)ADV_WARP_WORDS * 4; }
// Dynamic shared memory of the sweep for a grammar: per-warp scratch plus, if they fit the
// budget, the item-info / byte-class / byte-class-number tables.
constexpr uint32_t SWEEP_SMEM_LIMIT = 224 * 1024;  // what the sweep kernels opt in to
void sweep_layout(const GrammarDev& G, uint32_t* smem_bytes, uint32_t* tables_in_smem) {
  const uint32_t ntw = (2u * G.Nw + 7u) & ~7u;
  const uint32_t warp_words = SWEEP_CUR + SWEEP_HSET + ntw + W_CTRS + 8;
  uint32_t bytes = SWEEP_WARPS * warp_words * 4u;
  const uint32_t tab = G.hot_words * 4u;
  *tables_in_smem = (tab <= HOT_TABLE_BYTES && bytes + tab <= SWEEP_SMEM_LIMIT) ? 1u : 0u;
  if (*tables_in_smem) bytes += tab;
  *smem_bytes = bytes;
}
int sweep_warps() { return SWEEP_WARPS; }

cudaError_t configure_kernels() {
  cudaError_t e;
  if ((e = opt_in_smem((const void*)init_kernel, init_smem_bytes())) != cudaSuccess) return e;
  if ((e = opt_in_smem((const void*)advance_kernel, (size_t)ADV_WARPS * ADV_WARP_WORDS * 4 + HOT_TABLE_BYTES)) != cudaSuccess) return e;
  if ((e = opt_in_smem((const void*)forced_kernel, (size_t)ADV_WARPS * ADV_WARP_WORDS * 4 + HOT_TABLE_BYTES)) != cudaSuccess) return e;
  if ((e = opt_in_smem((const void*)sweep_kernel, SWEEP_SMEM_LIMIT)) != cudaSuccess) return e;
  return configure_walk_kernels();
}

cudaError_t sweep_blocks_per_sm(int* out, uint32_t smem_bytes) {
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(out, sweep_kernel, SWEEP_WARPS * 32, smem_bytes);
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
void launch_forced(const GrammarDev& G, const StateDev& S, uint8_t* bytes_out, size_t stride, uint32_t* len_out,
                   uint32_t max_len, cudaStream_t st) {
  forced_kernel<<<(S.B + ADV_WARPS - 1) / ADV_WARPS, ADV_WARPS * 32, adv_smem_bytes(G), st>>>(G, S, bytes_out, stride, len_out, max_len);
}
void launch_advance(const GrammarDev& G, const StateDev& S, const int32_t* tokens, int32_t* status, cudaStream_t st) {
  advance_kernel<<<(S.B + ADV_WARPS - 1) / ADV_WARPS, ADV_WARPS * 32, adv_smem_bytes(G), st>>>(G, S, tokens, status);
}
static void launch_sweep_coop(const GrammarDev& G, const StateDev& S, int grid, cudaStream_t st) {
  GrammarDev g = G;
  StateDev s = S;
  void* args[] = {&g, &s};
  cudaLaunchCooperativeKernel((const void*)sweep_kernel, dim3((unsigned)grid), dim3(SWEEP_WARPS * 32), args,
                              S.au.smem_bytes, st);
}
void launch_plan(const GrammarDev& G, const StateDev& S, cudaStream_t st) { plan_kernel<<<1, 1024, 0, st>>>(G, S); }
void launch_publish(const StateDev& S, cudaStream_t st) { publish_kernel<<<(S.B + 255) / 256, 256, 0, st>>>(S); }
// the sweep alone, for jobs the caller has already listed (used by the allocation-free entry point)
void launch_sweep(const GrammarDev& G, const StateDev& S, int grid, cudaStream_t st) { launch_sweep_coop(G, S, grid, st); }
void launch_gather(const GrammarDev& G, const StateDev& S, uint32_t* out, size_t stride_words, cudaStream_t st) {
  dim3 grid((unsigned)std::min<size_t>((stride_words + 255) / 256, 64), S.B);
  gather_kernel<<<grid, 256, 0, st>>>(G, S, out, stride_words);
}
void launch_apply(const uint32_t* mask, size_t stride_words, void* logits, int dtype, uint32_t batch, uint32_t V,
                  size_t row_stride, cudaStream_t st) {
  if (batch == 0 || V == 0) return;
  dim3 grid((unsigned)std::max<uint32_t>(1u, std::min<uint32_t>((V / 8 + 1023) / 1024, 64)), batch);
  if (dtype == FMT_BF16) apply_kernel<uint16_t><<<grid, 256, 0, st>>>(mask, stride_words, (uint16_t*)logits, V, row_stride);
  else apply_kernel<uint32_t><<<grid, 256, 0, st>>>(mask, stride_words, (uint32_t*)logits, V, row_stride);
}
void launch_gather_apply(const GrammarDev& G, const StateDev& S, void* logits, int dtype, size_t row_stride,
                         uint32_t* mask_out, size_t stride_words, cudaStream_t st) {
  dim3 grid((unsigned)std::max<uint32_t>(1u, std::min<uint32_t>((G.V / 8 + 1023) / 1024, 64)), S.B);  // about four groups of 8 tokens per thread
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
void launch_survivors(const GrammarDev& G, const StateDev& Old, const StateDev& S, const uint32_t* old_count, cudaStream_t st) {
  const uint32_t n = Old.max_states;
  dim3 grid((n + 255) / 256, 256);
  survivors_kernel<<<grid, 32, 0, st>>>(G, Old, S, old_count);
}
void launch_query(const StateDev& S, uint8_t* a, uint8_t* f, uint32_t* ns, uint32_t* ni, int32_t* sid, cudaStream_t st) {
  query_kernel<<<(S.B + 127) / 128, 128, 0, st>>>(S, a, f, ns, ni, sid);
}

}  // namespace fmt
