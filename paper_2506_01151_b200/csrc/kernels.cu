// CUDA kernels of the mask path (sm_100a): advance, plan / sweep / publish of the mask fill, gather
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

constexpr uint32_t HOT_TABLE_BYTES = 24 * 1024;  // grammar tables up to this size are staged in shared memory

__global__ void __launch_bounds__(ADV_WARPS * 32) advance_kernel(GrammarDev Gg, StateDev S, const int32_t* tokens,
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
  if (r == 0) return finish(FMT_ERR_TOKEN_REJECTED);
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

// One block decides, row by row, where each mask comes from: the state cache, another row of
// this call with the same chart, or a fresh computation (a "job").
__global__ void __launch_bounds__(1024) plan_kernel(GrammarDev G, StateDev S) {
  if (threadIdx.x == 0) {
    S.counters[CNT_N_JOBS] = 0u;
    S.counters[CNT_AUTO_ITEMS] = 0u;
    S.counters[CNT_JOB_NEXT] = 0u;
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
}

// ===================================================================================== fill: sweep

}  // namespace fmt
#include "sweep_cta.cuh"
namespace fmt {

// Publish the masks computed in this call to the cache (or release the claim when the row had
// no cache row, or broke).
__global__ void publish_kernel(StateDev S) {
  const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t n_jobs = S.counters[CNT_N_JOBS];
  if (j < n_jobs) {
    const uint32_t row = S.jobs[j];
    const int32_t sid = S.row_state[row];
    const bool broken = (S.row_flags[row] & ROW_BROKEN) != 0u;
    if (sid >= 0) {
      const int32_t mrow = S.row_mask[row];
      S.st_mask[sid] = (!broken && mrow >= (int32_t)S.B) ? mrow : -1;
    }
  }
}

__device__ __forceinline__ int32_t resolve_mask_row(const StateDev& S, uint32_t row) {
  int32_t r = S.row_mask[row];
  if (r <= MASK_ALIAS0) r = S.row_mask[(uint32_t)(MASK_ALIAS0 - r)];
  if (S.row_flags[row] & ROW_BROKEN) r = MASK_ZERO;
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

// logits[t] = -inf where bit t is 0, for one row.  Each thread takes one mask word (32 tokens:
// 64 bytes of bf16, 128 bytes of fp32) at a time and handles it in groups of 8 tokens with 16-byte
// accesses when the row is 16-byte aligned, else token by token.  Groups whose 8 tokens are all
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
  for (uint32_t wd = tid; wd < words; wd += nthreads) {
    uint32_t word = 0;
    if (mask_row) word = __ldg(&mask_row[wd]);
    else if (special == MASK_EOS_ONLY && eos >= 0 && wd == ((uint32_t)eos >> 5)) word = 1u << ((uint32_t)eos & 31u);
    if (mask_out) mask_out[wd] = word;
    if (word == 0xFFFFFFFFu) continue;
    const uint32_t t0 = wd * 32;
    if (aligned && t0 + 32 <= V) {
#pragma unroll
      for (uint32_t gq = 0; gq < 4; ++gq) {
        const uint32_t bits = (word >> (8 * gq)) & 0xFFu;
        if (bits != 0xFFu) apply_group<T>(logits + t0 + 8 * gq, bits);
      }
    } else {
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

static size_t adv_smem_bytes(const GrammarDev& G) {
  return (size_t)ADV_WARPS * ADV_WARP_WORDS * 4 + (G.hot_words * 4u <= HOT_TABLE_BYTES ? G.hot_words * 4u : 0u);
}
static size_t init_smem_bytes() { return (size_t)ADV_WARP_WORDS * 4; }
// Decide what of a sweep CTA's working set lives in shared memory for this grammar and fill in
// the layout fields of `A` (cap must be set): the grammar's hot tables and the mask row when they
// are small enough, a staged base chart, and as many automaton records and item words as the
// rest of the budget holds.
void sweep_plan(const GrammarDev& G, AutoDev& A) {
  A.rec_words = (AR_TRANS + (G.n_eq + 1u) / 2u + 3u) & ~3u;
  A.tables_in_smem = G.hot_words * 4u <= HOT_TABLE_BYTES ? 1u : 0u;
  A.mask_in_smem = G.Wm * 4u <= 48u * 1024u ? 1u : 0u;
  A.chart_sm_words = SW_CHART_SM;
  A.level_pad = (G.max_level + 63u) & ~63u;
  A.sm_states = 0;
  A.sm_items = 0;
  const uint32_t budget = SW_SMEM_BUDGET / 4u;
  uint32_t fixed = sweep_smem(G, A).total;
  if (fixed + 4096u > budget && A.mask_in_smem) {  // a huge vocabulary: assemble the mask row in global memory
    A.mask_in_smem = 0;
    fixed = sweep_smem(G, A).total;
  }
  const uint32_t rest = budget > fixed + 64u ? budget - fixed - 64u : 0u;
  A.sm_items = std::min(rest / 3u, 16384u) & ~3u;
  A.sm_states = std::min(std::min((rest - A.sm_items) / A.rec_words, A.cap), AUTO_MAX_STATES);
  if (A.sm_states < 1u) A.sm_states = 0u, A.sm_items = 0u;
  A.smem_bytes = sweep_smem(G, A).total * 4u;
}
int sweep_warps() { return SW_WARPS; }

cudaError_t configure_kernels() {
  cudaError_t e;
  if ((e = opt_in_smem((const void*)init_kernel, init_smem_bytes())) != cudaSuccess) return e;
  if ((e = opt_in_smem((const void*)advance_kernel, (size_t)ADV_WARPS * ADV_WARP_WORDS * 4 + HOT_TABLE_BYTES)) != cudaSuccess) return e;
  if ((e = opt_in_smem((const void*)sweep_kernel, SW_SMEM_BUDGET)) != cudaSuccess) return e;
  return cudaSuccess;
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
  advance_kernel<<<(S.B + ADV_WARPS - 1) / ADV_WARPS, ADV_WARPS * 32, adv_smem_bytes(G), st>>>(G, S, tokens, status);
}
void launch_sweep(const GrammarDev& G, const StateDev& S, cudaStream_t st) {
  sweep_kernel<<<S.au.grid, SW_THREADS, S.au.smem_bytes, st>>>(G, S);
}
void launch_fill(const GrammarDev& G, const StateDev& S, cudaStream_t st, cudaEvent_t before_sweep, cudaEvent_t after_sweep) {
  plan_kernel<<<1, 1024, 0, st>>>(G, S);
  if (before_sweep) cudaEventRecord(before_sweep, st);
  launch_sweep(G, S, st);
  if (after_sweep) cudaEventRecord(after_sweep, st);
  publish_kernel<<<(S.B + 255) / 256, 256, 0, st>>>(S);
}
void launch_gather(const GrammarDev& G, const StateDev& S, uint32_t* out, size_t stride_words, cudaStream_t st) {
  dim3 grid((unsigned)std::min<size_t>((stride_words + 255) / 256, 64), S.B);
  gather_kernel<<<grid, 256, 0, st>>>(G, S, out, stride_words);
}
void launch_apply(const uint32_t* mask, size_t stride_words, void* logits, int dtype, uint32_t batch, uint32_t V,
                  size_t row_stride, cudaStream_t st) {
  if (batch == 0 || V == 0) return;
  dim3 grid((unsigned)std::min<uint32_t>(((V + 31) / 32 + 255) / 256, 64), batch);
  if (dtype == FMT_BF16) apply_kernel<uint16_t><<<grid, 256, 0, st>>>(mask, stride_words, (uint16_t*)logits, V, row_stride);
  else apply_kernel<uint32_t><<<grid, 256, 0, st>>>(mask, stride_words, (uint32_t*)logits, V, row_stride);
}
void launch_gather_apply(const GrammarDev& G, const StateDev& S, void* logits, int dtype, size_t row_stride,
                         uint32_t* mask_out, size_t stride_words, cudaStream_t st) {
  dim3 grid((unsigned)std::min<uint32_t>(((G.V + 31) / 32 + 255) / 256, 64), S.B);
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
