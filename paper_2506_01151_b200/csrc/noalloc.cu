// fmt_fill_mask_noalloc: the trie sweep for callers that may not allocate device memory.
//
// All scratch the sweep needs lives in one file-scope __device__ array that is part of the
// library image.  Host code must not pass the array's name to a kernel (on the host it is only
// a stand-in symbol): the device address is looked up once per device with
// cudaGetSymbolAddress and passed as an ordinary pointer.
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>

#include "../../include/fmt.h"
#include "device_tables.h"
#include "kernels.h"

namespace {

using namespace fmt;

constexpr uint32_t NA_MAX = FMT_NOALLOC_MAX_CHARTS;
constexpr uint32_t NA_GRID = 12;            // CTAs of the sweep
constexpr uint32_t NA_ARENA_ITEMS = 8192;   // per-warp overflow area for Earley sets (items)
constexpr uint32_t NA_HSET_SLOTS = 2048;    // per-warp overflow uniqueness hash
// header: counters, then per-chart arrays
constexpr uint32_t NA_OFF_COUNTERS = 0;                          // [CNT_TOTAL]
constexpr uint32_t NA_OFF_JOBS = 256;                            // [NA_MAX]
constexpr uint32_t NA_REQ_CAP = 1u << 16;                        // transitions queued per trie depth
constexpr uint32_t NA_OFF_FLAGS = NA_OFF_JOBS + NA_MAX;          // [NA_MAX]
constexpr uint32_t NA_OFF_MASKROW = NA_OFF_FLAGS + NA_MAX;       // [NA_MAX] int32
constexpr uint32_t NA_OFF_CHART = NA_OFF_MASKROW + NA_MAX;       // [NA_MAX] uint64 (8-byte aligned)
constexpr uint32_t NA_OFF_BAD = NA_OFF_CHART + 2 * NA_MAX;       // [NA_MAX] header check failed
constexpr uint32_t NA_OFF_NSTATES = NA_OFF_BAD + NA_MAX;         // [NA_MAX] Earley sets created per chart
constexpr uint32_t NA_OFF_JOBINFO = NA_OFF_NSTATES + NA_MAX;     // [NA_MAX] uint4 (16-byte aligned)
constexpr uint32_t NA_HEADER_WORDS = 1024;
constexpr size_t NA_WARPS = (size_t)NA_GRID * SWEEP_WARPS;
constexpr size_t NA_BIG_WORDS = NA_WARPS * (NA_ARENA_ITEMS + NA_HSET_SLOTS);
// the sweep's tables of Earley sets: per chart 64 Ki words of records and 2048 hash slots, and one
// pool of 2 Mi item words for all charts of a call
constexpr uint32_t NA_REC_WORDS_PER_CHART = 65536;
constexpr uint32_t NA_HASH_SLOTS = 2048;
constexpr uint32_t NA_ITEM_WORDS = 2u << 20;
constexpr size_t NA_OFF_BIG = NA_HEADER_WORDS;
constexpr size_t NA_OFF_RECS = NA_OFF_BIG + NA_BIG_WORDS;
constexpr size_t NA_OFF_HASH = NA_OFF_RECS + (size_t)NA_MAX * NA_REC_WORDS_PER_CHART;
constexpr size_t NA_OFF_ITEMS = NA_OFF_HASH + (size_t)NA_MAX * NA_HASH_SLOTS;
// per (chart, trie node) one uint16: which Earley set the node's bytes lead to
constexpr size_t NA_ST_ENTRIES = 8u << 20;
constexpr size_t NA_OFF_ST = NA_OFF_ITEMS + NA_ITEM_WORDS;
constexpr size_t NA_OFF_REQ = NA_OFF_ST + NA_ST_ENTRIES / 2;       // 8-byte aligned: all sizes above are even
constexpr size_t NA_WORDS = NA_OFF_REQ + 2 * (size_t)NA_REQ_CAP;
static_assert(CNT_TOTAL <= NA_OFF_JOBS, "the counters overlap the job list");
static_assert(NA_OFF_JOBINFO + 4 * NA_MAX <= NA_HEADER_WORDS, "header too small");
static_assert((NA_OFF_JOBINFO % 4) == 0, "job records must be 16-byte aligned");
static_assert((NA_OFF_CHART % 2) == 0, "64-bit offsets must be 8-byte aligned");

// ~55 MB, held by every GPU that loads the library until the process exits
static __device__ __align__(256) uint32_t g_noalloc_scratch[NA_WORDS];

struct Offsets {
  uint64_t v[NA_MAX + 1];
};

// Fill the header for this call, check each chart's header against its slot, zero the output
// masks (setting the EOS bit of accepting charts) and clear the overflow hashes, which must be
// all-empty before the sweep and may hold anything after an earlier call that broke off.
__global__ void noalloc_prepare_kernel(GrammarDev G, StateDev S, uint32_t* scratch, const uint32_t* charts, Offsets off,
                                       uint32_t n, uint32_t* mask) {
  const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t nth = (size_t)gridDim.x * blockDim.x;
  if (tid < CNT_TOTAL) S.counters[tid] = 0u;  // (the sweep's generation is 1 in every call: the hashes and the queue are cleared below)
  if (tid < n) {
    const uint32_t r = (uint32_t)tid;
    const uint32_t* ch = charts + off.v[r];
    const uint64_t room = off.v[r + 1] - off.v[r];
    bool ok = room >= CH_HDR + 2;
    if (ok) {
      const uint64_t m = ch[CH_SETS], items = ch[CH_ITEMS], words = ch[CH_WORDS];
      ok = m >= 1 && words <= room && words == CH_HDR + m + 1 + items && ch[CH_HDR + m] == items;
    }
    scratch[NA_OFF_BAD + r] = ok ? 0u : 1u;
    S.row_chart[r] = off.v[r];
    S.row_mask[r] = (int32_t)r;
    S.row_flags[r] = 0u;
  }
  for (size_t i = tid; i < (size_t)n * G.Wm; i += nth) mask[i] = 0u;
  for (size_t i = tid; i < (size_t)NA_MAX * NA_HASH_SLOTS; i += nth) S.au.hash[i] = 0u;
  for (size_t i = tid; i < NA_REQ_CAP; i += nth) S.au.req[i] = 0ull;  // no stale tags: every call is generation 1
  uint32_t* big = S.big_scratch;
  const size_t per_warp = (size_t)NA_ARENA_ITEMS + NA_HSET_SLOTS;
  for (size_t i = tid; i < NA_WARPS * NA_HSET_SLOTS; i += nth)
    big[(i / NA_HSET_SLOTS) * per_warp + NA_ARENA_ITEMS + (i % NA_HSET_SLOTS)] = 0xffffffffu;
}

// One CTA per chart whose header was accepted: the rest of the chart.  The sweep indexes its tables
// with what the chart says, so every word is checked here: the sets' offsets must not decrease, every
// item must name a dotted rule of this grammar and start in a set of this chart.
__global__ void noalloc_validate_kernel(GrammarDev G, uint32_t* scratch, const uint32_t* charts, Offsets off, uint32_t n) {
  const uint32_t r = blockIdx.x;
  if (r >= n || scratch[NA_OFF_BAD + r]) return;
  const uint32_t* ch = charts + off.v[r];
  const uint32_t m = ch[CH_SETS], items = ch[CH_ITEMS];
  const uint32_t* set_off = ch + CH_HDR;
  const uint32_t* it = set_off + m + 1;
  bool bad = false;
  for (uint32_t i = threadIdx.x; i < m; i += blockDim.x) {
    const uint32_t a = set_off[i], b = set_off[i + 1];
    if (a > b || b > items || (i == 0 && a != 0u)) bad = true;
  }
  for (uint32_t k = threadIdx.x; k < items; k += blockDim.x) {
    const uint32_t x = it[k];
    if ((x & 0xFFFFu) >= G.D || (x >> 16) >= m) bad = true;
  }
  if (bad) scratch[NA_OFF_BAD + r] = 1u;  // (every writer writes the same value)
}

// One thread: the job list holds the charts that passed both checks.
__global__ void noalloc_jobs_kernel(StateDev S, const uint32_t* scratch, uint32_t n) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  uint32_t j = 0;
  for (uint32_t r = 0; r < n; ++r)
    if (!scratch[NA_OFF_BAD + r]) S.jobs[j++] = r;
  S.counters[CNT_N_JOBS] = j;
}

__global__ void noalloc_finish_kernel(GrammarDev G, StateDev S, const uint32_t* scratch, uint32_t n, uint32_t* mask,
                                      int32_t* status) {
  const uint32_t r = blockIdx.x;
  if (r >= n) return;
  const bool bad = scratch[NA_OFF_BAD + r] != 0u;
  // a sweep that gave up on a wait leaves no mask to trust, whichever chart it was at
  const bool broken = (S.row_flags[r] & ROW_BROKEN) != 0u || S.counters[CNT_BAR_ERR] != 0u;
  if (broken)
    for (uint32_t i = threadIdx.x; i < G.Wm; i += blockDim.x) mask[(size_t)r * G.Wm + i] = 0u;
  if (status && threadIdx.x == 0) status[r] = bad ? FMT_ERR_INVALID_ARG : (broken ? FMT_ERR_CAPACITY : FMT_OK);
}

// per-device set-up, done by the first call on that device
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
uint32_t* g_scratch_addr[kMaxDevices] = {};

cudaError_t scratch_for_current_device(int dev, uint32_t** out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    uint32_t* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    e = configure_kernels();  // raises the dynamic shared-memory limit of the sweep kernel on this device
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

fmt_status fail(fmt_status code, const char* msg) {
  set_last_error(msg);
  return code;
}

}  // namespace

extern "C" fmt_status fmt_fill_mask_noalloc(const fmt_grammar* g, const uint32_t* charts_dev,
                                            const uint64_t* chart_offsets, uint32_t n, uint32_t* mask_dev,
                                            int32_t* status_dev, void* stream) {
  if (!g || !charts_dev || !chart_offsets || !mask_dev) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  if (n == 0) return FMT_OK;
  if (n > NA_MAX) return fail(FMT_ERR_CAPACITY, "fmt_fill_mask_noalloc takes at most 64 charts per call");
  int gdev = -1, dev = -1;
  const GrammarDev* G = grammar_device_tables(g, &gdev);
  if (!G) return fail(FMT_ERR_INVALID_ARG, "the grammar was compiled host_only");
  if (cudaGetDevice(&dev) != cudaSuccess || dev != gdev || dev < 0 || dev >= kMaxDevices)
    return fail(FMT_ERR_INVALID_ARG, "the grammar belongs to another device than the current one");
  const size_t st_stride = ((size_t)G->T + 63u) & ~(size_t)63u;
  if ((size_t)n * st_stride > NA_ST_ENTRIES)
    return fail(FMT_ERR_CAPACITY,
                "fmt_fill_mask_noalloc: charts x trie nodes exceeds the built-in scratch (8 Mi entries); pass fewer charts per call");
  Offsets off;
  for (uint32_t r = 0; r <= n; ++r) {
    off.v[r] = chart_offsets[r];
    if (r && off.v[r] < off.v[r - 1]) return fail(FMT_ERR_INVALID_ARG, "chart_offsets must not decrease");
  }
  for (uint32_t r = n + 1; r <= NA_MAX; ++r) off.v[r] = off.v[n];
  uint32_t* scratch = nullptr;
  cudaError_t e = scratch_for_current_device(dev, &scratch);
  if (e != cudaSuccess) return fail(FMT_ERR_CUDA, cudaGetErrorString(e));

  StateDev S{};
  S.B = n;
  S.cache_on = 0;
  S.gen = 1;  // the hashes are cleared by every call
  S.arena = const_cast<uint32_t*>(charts_dev);  // the sweep only reads charts
  S.counters = scratch + NA_OFF_COUNTERS;
  S.jobs = scratch + NA_OFF_JOBS;
  S.row_flags = scratch + NA_OFF_FLAGS;
  S.row_mask = reinterpret_cast<int32_t*>(scratch + NA_OFF_MASKROW);
  S.row_chart = reinterpret_cast<uint64_t*>(scratch + NA_OFF_CHART);
  S.mask_rows = mask_dev;
  S.big_scratch = scratch + NA_OFF_BIG;
  S.big_arena_items = NA_ARENA_ITEMS;
  S.big_hset_slots = NA_HSET_SLOTS;
  S.au.rec_words = (AR_TRANS + G->n_eq + 31u) & ~31u;
  S.au.cap = std::min<uint32_t>(1024u, NA_REC_WORDS_PER_CHART / S.au.rec_words);
  S.au.hash_mask = NA_HASH_SLOTS - 1;
  S.au.items_cap = NA_ITEM_WORDS;
  S.au.recs = scratch + NA_OFF_RECS;
  S.au.hash = scratch + NA_OFF_HASH;
  S.au.items = scratch + NA_OFF_ITEMS;
  S.au.n_states = scratch + NA_OFF_NSTATES;
  S.au.st = reinterpret_cast<uint16_t*>(scratch + NA_OFF_ST);
  S.au.st_stride = (uint32_t)st_stride;
  S.au.req = reinterpret_cast<unsigned long long*>(scratch + NA_OFF_REQ);
  S.au.req_cap = NA_REQ_CAP;
  S.au.job_info = reinterpret_cast<uint4*>(scratch + NA_OFF_JOBINFO);
  sweep_layout(*G, &S.au.smem_bytes, &S.au.tables_in_smem);
  cudaStream_t st = (cudaStream_t)stream;
  noalloc_prepare_kernel<<<256, 256, 0, st>>>(*G, S, scratch, charts_dev, off, n, mask_dev);
  noalloc_validate_kernel<<<n, 256, 0, st>>>(*G, scratch, charts_dev, off, n);
  noalloc_jobs_kernel<<<1, 32, 0, st>>>(S, scratch, n);
  launch_sweep(*G, S, (int)NA_GRID, st);
  noalloc_finish_kernel<<<n, 128, 0, st>>>(*G, S, scratch, n, mask_dev, status_dev);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(FMT_ERR_CUDA, cudaGetErrorString(e));
  return FMT_OK;
}
