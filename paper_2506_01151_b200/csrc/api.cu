// The C-ABI of include/fmt.h: handle management, uploads and kernel launches.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/fmt.h"
#include "device_tables.h"
#include "host_tables.h"
#include "kernels.h"

using namespace fmt;

namespace {

thread_local std::string g_last_error;

fmt_status fail(fmt_status code, const std::string& msg) {
  g_last_error = msg;
  return code;
}
fmt_status cuda_fail(cudaError_t e, const char* what) {
  return fail(e == cudaErrorMemoryAllocation ? FMT_ERR_OOM : FMT_ERR_CUDA,
              std::string(what) + ": " + cudaGetErrorString(e));
}

struct DeviceBuffers {
  std::vector<void*> ptrs;
  size_t bytes = 0;
  ~DeviceBuffers() {
    for (void* p : ptrs) cudaFree(p);
  }
  template <typename T>
  cudaError_t upload(const std::vector<T>& v, const T** out) {
    void* p = nullptr;
    size_t bytes = std::max<size_t>(v.size() * sizeof(T), 16);
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) return e;
    ptrs.push_back(p);
    if (!v.empty()) {
      e = cudaMemcpy(p, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice);
      if (e != cudaSuccess) return e;
    }
    *out = static_cast<const T*>(p);
    return cudaSuccess;
  }
  template <typename T>
  cudaError_t alloc(size_t count, T** out, int fill_byte) {
    void* p = nullptr;
    size_t bytes = std::max<size_t>(count * sizeof(T), 16);
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) return e;
    ptrs.push_back(p);
    this->bytes += bytes;
    e = cudaMemset(p, fill_byte, bytes);
    if (e != cudaSuccess) return e;
    *out = static_cast<T*>(p);
    return cudaSuccess;
  }
};

}  // namespace

struct fmt_grammar {
  HostTables host;
  GrammarDev dev{};
  bool on_device = false;
  int device = -1;
  DeviceBuffers bufs;
};

// CUDA-event pairs around the four kinds of work, filled while profiling is enabled.
struct Profiler {
  static constexpr size_t kMaxPairs = 16384;
  bool on = false;
  std::vector<cudaEvent_t> a[4], b[4];  // 0 advance, 1 trie sweep of the fill, 2 logits masking, 3 the fill's work on roots
  size_t used[4] = {0, 0, 0, 0};
  bool next(int kind, cudaEvent_t* before, cudaEvent_t* after) {
    *before = *after = nullptr;
    if (!on || used[kind] >= kMaxPairs) return false;
    if (used[kind] == a[kind].size()) {
      cudaEvent_t x, y;
      if (cudaEventCreate(&x) != cudaSuccess) return false;
      if (cudaEventCreate(&y) != cudaSuccess) {
        cudaEventDestroy(x);
        return false;
      }
      a[kind].push_back(x);
      b[kind].push_back(y);
    }
    *before = a[kind][used[kind]];
    *after = b[kind][used[kind]];
    ++used[kind];
    return true;
  }
  ~Profiler() {
    for (int k = 0; k < 4; ++k) {
      for (auto e : a[k]) cudaEventDestroy(e);
      for (auto e : b[k]) cudaEventDestroy(e);
    }
  }
};

struct fmt_state {
  Profiler prof;
  const fmt_grammar* g = nullptr;
  StateDev dev{};
  DeviceBuffers bufs;
  int32_t* init_state_dev = nullptr;
  int32_t* result_dev = nullptr;
  uint8_t* query_dev = nullptr;  // scratch for fmt_state_query
  int sweep_grid = 1;
  uint32_t next_gen = 1;      // generations handed to the fills: two per fill, 1 .. 65534
  size_t device_bytes = 0;    // what fmt_state_create allocated
  // The device sets this host-mapped word when the state cache has no room for a new entry; the next
  // fmt_state_advance empties the cache (all entries at once) and caching goes on.
  // Two generations of cache storage (chart pool, per-entry tables, mask rows): emptying the cache switches to
  // the other one and carries over the entries that were found again after they were made.
  int generation = 0;
  uint64_t* st_off2[2] = {nullptr, nullptr};
  int32_t* st_mask2[2] = {nullptr, nullptr};
  uint8_t* st_ref2[2] = {nullptr, nullptr};
  uint64_t pool_base2[2] = {0, 0};
  uint32_t mrow_base2[2] = {0, 0};
  uint32_t* old_count_dev = nullptr;
  uint64_t survivors_runs = 0;
  uint32_t* full_flag_host = nullptr;
  bool skip_full_check = false;
  uint64_t flushes = 0;
  ~fmt_state() {
    if (full_flag_host) cudaFreeHost(full_flag_host);
  }
};

// Two fresh generations for a fill (its root sweep and its walk).  Tables tagged with a generation
// are never cleared between fills; when the 16-bit numbers start over they all are.
static cudaError_t next_generations(fmt_state* s, cudaStream_t st) {
  StateDev& d = s->dev;
  cudaError_t e = cudaSuccess;
  if (s->next_gen + 1u > 65534u) {
    e = cudaMemsetAsync(d.au.hash, 0, (size_t)d.B * (d.au.hash_mask + 1u) * 4, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(d.au.req, 0, (size_t)d.au.req_cap * 8, st);
    if (e == cudaSuccess && d.rt.on) e = cudaMemsetAsync(d.cx.ctab, 0, (size_t)d.B * CT_SLOTS * 8, st);
    if (e == cudaSuccess && d.rt.on) e = cudaMemsetAsync(d.cx.req2, 0, (size_t)d.cx.req2_cap * 16, st);
    s->next_gen = 1;
  }
  d.gen = s->next_gen;
  d.gen_ctx = s->next_gen + 1u;
  s->next_gen += 2u;
  return e;
}

namespace fmt {
const GrammarDev* grammar_device_tables(const ::fmt_grammar* g, int* device) {
  if (!g || !g->on_device) return nullptr;
  if (device) *device = g->device;
  return &g->dev;
}
void set_last_error(const char* msg) { g_last_error = msg; }
}  // namespace fmt

extern "C" {

const char* fmt_last_error(void) { return g_last_error.c_str(); }

fmt_status fmt_compile(const char* ebnf, size_t ebnf_len, const char* start_rule, const uint8_t* vocab_bytes,
                       const uint64_t* vocab_offsets, uint32_t V, int32_t eos_token_id, const fmt_compile_options* opt,
                       fmt_grammar** out) {
  if (!out) return fail(FMT_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (!ebnf || !start_rule || !vocab_offsets || (!vocab_bytes && V > 0 && vocab_offsets[V] > vocab_offsets[0]))
    return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  if (V == 0) return fail(FMT_ERR_INVALID_ARG, "the vocabulary is empty");
  if (eos_token_id < -1 || eos_token_id >= (int64_t)V) return fail(FMT_ERR_INVALID_ARG, "eos_token_id out of range");
  fmt_grammar* g = new (std::nothrow) fmt_grammar;
  if (!g) return fail(FMT_ERR_OOM, "out of host memory");
  try {
    compile_grammar(ebnf, ebnf_len, start_rule, g->host, !(opt && opt->no_dfa_terminals));
    static const uint8_t none = 0;
    build_trie(vocab_bytes ? vocab_bytes : &none, vocab_offsets, V, eos_token_id, g->host);
    if (eos_token_id >= 0 && vocab_offsets[eos_token_id + 1] != vocab_offsets[eos_token_id])
      throw CompileError{FMT_ERR_INVALID_ARG, "the EOS token must have no bytes"};
  } catch (const CompileError& e) {
    delete g;
    return fail((fmt_status)e.code, e.msg);
  } catch (const std::bad_alloc&) {
    delete g;
    return fail(FMT_ERR_OOM, "out of host memory");
  }
  if (!(opt && opt->host_only)) {
    const HostTables& h = g->host;
    GrammarDev& d = g->dev;
    d.D = h.D, d.N = h.N, d.C = h.C, d.Nw = h.Nw;
    d.V = h.V, d.Wm = h.Wm, d.T = h.T, d.depth = h.depth;
    d.eos = h.eos;
    d.start_nullable = h.start_nullable ? 1u : 0u;
    cudaError_t e = cudaGetDevice(&g->device);
#define UP(field) if (e == cudaSuccess) e = g->bufs.upload(h.field, &d.field)
    UP(lhs);
    d.n_eq = h.n_eq;
    {  // info | class_bits | eq_of_byte | nt_closure | direct_off | direct_items, each 16-byte aligned
      std::vector<uint32_t> blob;
      auto put = [&](const void* src, size_t bytes) {
        size_t at = blob.size();
        blob.resize(at + ((bytes + 15) / 16) * 4, 0u);
        memcpy(blob.data() + at, src, bytes);
        return at;
      };
      const size_t o_info = put(h.info.data(), h.info.size() * 4);
      const size_t o_cls = put(h.class_bits.data(), h.class_bits.size() * 4);
      const size_t o_eq = put(h.eq_of_byte.data(), 256);
      const size_t o_clo = put(h.nt_closure.data(), h.nt_closure.size() * 4);
      const size_t o_doff = put(h.direct_off.data(), h.direct_off.size() * 4);
      const size_t o_dit = put(h.direct_items.data(), h.direct_items.size() * 2);
      if (e == cudaSuccess) e = g->bufs.upload(blob, &d.hot_block);
      d.hot_words = (uint32_t)blob.size();
      d.info = d.hot_block + o_info;
      d.class_bits = d.hot_block + o_cls;
      d.eq_of_byte = reinterpret_cast<const uint8_t*>(d.hot_block + o_eq);
      d.nt_closure = d.hot_block + o_clo;
      d.direct_off = d.hot_block + o_doff;
      d.direct_items = reinterpret_cast<const uint16_t*>(d.hot_block + o_dit);
    }
    d.dfa_first = h.dfa_first;
    if (h.dfa_states) {
      UP(dfa_trans);
      UP(dfa_done);
      UP(dfa_scan);
    }
    UP(node_byte);
    UP(parent);
    UP(node_depth);
    UP(lvl_off);
    UP(tok_node);
    UP(child_off);
    UP(tok_off);
    UP(tok_ids);
    UP(vocab_off);
    UP(vocab_bytes);
#undef UP
    if (e != cudaSuccess) {
      fmt_status st = cuda_fail(e, "uploading the grammar tables");
      delete g;
      return st;
    }
    g->on_device = true;
  }
  *out = g;
  return FMT_OK;
}

void fmt_grammar_destroy(fmt_grammar* g) { delete g; }

fmt_status fmt_json_schema_to_ebnf(const char* schema, size_t schema_len, char* out, size_t cap_bytes, size_t* size_bytes) {
  if (!schema || !size_bytes) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  try {
    const std::string text = json_schema_to_ebnf(schema, schema_len);
    *size_bytes = text.size();
    if (out && cap_bytes) memcpy(out, text.data(), std::min(text.size(), cap_bytes));
  } catch (const CompileError& e) {
    return fail((fmt_status)e.code, e.msg);
  } catch (const std::bad_alloc&) {
    return fail(FMT_ERR_OOM, "out of host memory");
  }
  return FMT_OK;
}

fmt_status fmt_compile_json_schema(const char* schema, size_t schema_len, const uint8_t* vocab_bytes,
                                   const uint64_t* vocab_offsets, uint32_t V, int32_t eos_token_id,
                                   const fmt_compile_options* opt, fmt_grammar** out) {
  if (!out) return fail(FMT_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (!schema) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  std::string text;
  try {
    text = json_schema_to_ebnf(schema, schema_len);
  } catch (const CompileError& e) {
    return fail((fmt_status)e.code, e.msg);
  } catch (const std::bad_alloc&) {
    return fail(FMT_ERR_OOM, "out of host memory");
  }
  return fmt_compile(text.data(), text.size(), "root", vocab_bytes, vocab_offsets, V, eos_token_id, opt, out);
}

fmt_status fmt_grammar_get_info(const fmt_grammar* g, fmt_grammar_info* out) {
  if (!g || !out) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  const HostTables& h = g->host;
  out->n_nonterminals = h.N;
  out->n_rules = h.P;
  out->n_dotted = h.D;
  out->n_classes = h.C;
  out->n_nullable = h.n_nullable;
  out->vocab_size = h.V;
  out->mask_words = h.Wm;
  out->trie_nodes = h.T;
  out->trie_depth = h.depth;
  out->n_byte_classes = h.n_eq;
  out->n_empty_tokens = h.n_empty;
  out->start_nullable = h.start_nullable ? 1u : 0u;
  out->n_automata = (uint32_t)h.dfa_nt.size();
  out->n_automaton_states = h.dfa_states;
  return FMT_OK;
}

fmt_status fmt_grammar_automaton_match(const fmt_grammar* g, uint32_t k, const uint8_t* bytes, size_t len, int* accepted,
                                       char* name_out, size_t name_cap) {
  if (!g || !accepted || (!bytes && len)) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  const HostTables& h = g->host;
  if (k >= h.dfa_nt.size()) return fail(FMT_ERR_INVALID_ARG, "no such automaton");
  if (name_out && name_cap) {
    const std::string& nm = h.nt_names[h.dfa_nt[k]];
    const size_t n = std::min(nm.size(), name_cap - 1);
    memcpy(name_out, nm.data(), n);
    name_out[n] = 0;
  }
  uint32_t q = h.dfa_start[k];
  *accepted = 0;
  for (size_t i = 0; i < len; ++i) {
    const uint16_t t = h.dfa_trans[(size_t)q * h.n_eq + h.eq_of_byte[bytes[i]]];
    if (t == 0xFFFFu) return FMT_OK;
    q = t & 0x3FFFu;
  }
  *accepted = h.dfa_accept[q] ? 1 : 0;
  return FMT_OK;
}

fmt_status fmt_grammar_copy_table(const fmt_grammar* g, int which, void* out, size_t cap_bytes, size_t* size_bytes) {
  if (!g || !size_bytes) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  const HostTables& h = g->host;
  const void* src = nullptr;
  size_t n = 0;
  switch (which) {
    case 0: src = h.child_off.data(), n = (size_t)(h.T + 1) * 4; break;
    case 1: src = h.node_byte.data(), n = h.T; break;
    case 2: src = h.parent.data(), n = (size_t)h.T * 4; break;
    case 3: src = h.tok_off.data(), n = (size_t)(h.T + 1) * 4; break;
    case 4: src = h.tok_ids.data(), n = (size_t)h.tok_off[h.T] * 4; break;
    case 5: src = h.lvl_off.data(), n = h.lvl_off.size() * 4; break;
    case 6: src = h.nullable.data(), n = h.N; break;
    case 7: src = h.info.data(), n = (size_t)h.D * 4; break;
    case 8: src = h.lhs.data(), n = (size_t)h.D * 2; break;
    case 9: src = h.tok_node.data(), n = h.tok_node.size() * 4; break;
    case 10: src = h.eq_of_byte.data(), n = 256; break;
    case 11: src = h.dfa_trans.data(), n = h.dfa_trans.size() * 2; break;
    case 12: src = h.dfa_accept.data(), n = h.dfa_accept.size(); break;
    case 13: src = h.dfa_start.data(), n = h.dfa_start.size() * 4; break;
    default: return fail(FMT_ERR_INVALID_ARG, "unknown table");
  }
  *size_bytes = n;
  if (out && cap_bytes) memcpy(out, src, std::min(n, cap_bytes));
  return FMT_OK;
}

fmt_status fmt_state_create(const fmt_grammar* g, uint32_t batch, const fmt_state_options* opt, void* stream,
                            fmt_state** out) {
  if (!out) return fail(FMT_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (!g || batch == 0) return fail(FMT_ERR_INVALID_ARG, "NULL grammar or empty batch");
  if (!g->on_device) return fail(FMT_ERR_INVALID_ARG, "the grammar was compiled host_only");
  if (batch > 65535) return fail(FMT_ERR_INVALID_ARG, "batch above 65535");
  cudaStream_t st = (cudaStream_t)stream;
  fmt_state* s = new (std::nothrow) fmt_state;
  if (!s) return fail(FMT_ERR_OOM, "out of host memory");
  s->g = g;
  StateDev& d = s->dev;
  d.B = batch;
  d.cache_on = (opt && opt->cache_disable) ? 0u : 1u;
  d.chart_words = (opt && opt->chart_words) ? opt->chart_words : 65536u;
  if (d.chart_words < 1024) d.chart_words = 1024;
  d.max_states = (opt && opt->max_states) ? opt->max_states : 262144u;
  d.max_mask_rows = (opt && opt->max_mask_rows) ? opt->max_mask_rows : 32768u;
  d.pool_words = (opt && opt->pool_words) ? opt->pool_words : (192ull << 20);
  if (!d.cache_on) {
    d.max_states = 1;
    d.max_mask_rows = 0;
    d.pool_words = 32;
  }
  uint32_t ht = 1024;
  while (ht < d.max_states * 2u) ht <<= 1;
  d.ht_mask = ht - 1;
  d.init_off = (uint64_t)batch * 3u * d.chart_words;
  d.pool_base = d.init_off + d.chart_words;
  d.pool_lo = d.pool_base;
  const bool two_gens = d.cache_on && !(opt && opt->cache_keep_when_full);
  s->pool_base2[0] = d.pool_base;
  s->pool_base2[1] = d.pool_base + (two_gens ? d.pool_words : 0);
  s->mrow_base2[0] = batch;
  s->mrow_base2[1] = batch + (two_gens ? d.max_mask_rows : 0);
  d.mrow_base = batch;
  d.big_arena_items = 1u << 16;
  d.big_hset_slots = 1u << 14;
  AutoDev& au = d.au;
  au.cap = (opt && opt->sweep_states) ? opt->sweep_states : std::min(32768u, std::max(2048u, (4u << 20) / batch));
  if (au.cap < 16) au.cap = 16;
  if (au.cap > 60000) au.cap = 60000;
  au.rec_words = (AR_TRANS + g->dev.n_eq + 31u) & ~31u;
  uint32_t hs = 64;
  while (hs < au.cap * 2u) hs <<= 1;
  au.hash_mask = hs - 1;
  au.items_cap = 128u << 20;
  d.poll_limit_shift = (opt && opt->wait_limit_log2) ? std::min(opt->wait_limit_log2, 30u) : 0u;
  RootDev& rt = d.rt;
  rt.on = (opt && opt->roots_enable) ? 1u : 0u;
  rt.max_roots = (opt && opt->max_roots) ? opt->max_roots : 4096u;
  rt.max_items = (opt && opt->root_max_items) ? std::min(opt->root_max_items, 1024u) : 1024u;
  rt.max_ph = (opt && opt->root_max_origins) ? std::min(opt->root_max_origins, 1024u) : 16u;
  uint32_t rh = 256;
  while (rh < rt.max_roots * 4u) rh <<= 1;
  rt.hash_mask = rh - 1;
  rt.charts_cap = rt.max_roots * 512u;
  rt.st_cap = 8u << 20;
  rt.it_cap = 64u << 20;
  rt.tr_cap = 256u << 20;
  rt.pend_cap = 4096;

  sweep_layout(g->dev, &au.smem_bytes, &au.tables_in_smem);
  cudaError_t e = configure_kernels();
  int per_sm = 0, sms = 0, dev = 0;
  if (e == cudaSuccess) e = sweep_blocks_per_sm(&per_sm, au.smem_bytes);
  if (e == cudaSuccess) e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess && per_sm < 1) {
    delete s;
    return fail(FMT_ERR_CUDA, "the sweep kernel does not fit on this device");
  }
  s->sweep_grid = std::max(1, per_sm * sms);
  const size_t big_words = (size_t)s->sweep_grid * sweep_warps() * ((size_t)d.big_arena_items + d.big_hset_slots);
#define AL(ptr, count, fill) if (e == cudaSuccess) e = s->bufs.alloc((size_t)(count), &(ptr), (fill))
  AL(d.arena, d.pool_base + d.pool_words * (two_gens ? 2 : 1), 0);
  AL(d.row_chart, batch, 0);
  AL(d.row_buf, batch, 0xFF);
  AL(d.row_state, batch, 0xFF);
  AL(d.row_flags, batch, 0);
  AL(d.row_mask, batch, 0xFF);
  AL(d.ht, ht, 0);
  AL(s->st_off2[0], d.max_states, 0);
  AL(s->st_mask2[0], d.max_states, 0xFF);
  AL(s->st_ref2[0], d.max_states, 0);
  if (two_gens) {
    AL(s->st_off2[1], d.max_states, 0);
    AL(s->st_mask2[1], d.max_states, 0xFF);
    AL(s->st_ref2[1], d.max_states, 0);
  }
  AL(s->old_count_dev, 4, 0);
  d.st_off = s->st_off2[0], d.st_mask = s->st_mask2[0], d.st_ref = s->st_ref2[0];
  AL(d.mask_rows, ((size_t)batch + (size_t)d.max_mask_rows * (two_gens ? 2 : 1)) * g->dev.Wm, 0);
  uint32_t trn = 1024;
  while (trn < d.max_states * 4u) trn <<= 1;
  d.tr_mask = trn - 1;
  AL(d.tr_key, trn, 0);
  AL(d.tr_val, trn, 0x80);
  AL(d.jobs, batch, 0);
  AL(d.counters, CNT_TOTAL, 0);
  AL(d.big_scratch, big_words, 0xFF);
  AL(au.recs, (size_t)batch * au.cap * au.rec_words, 0);
  AL(au.hash, (size_t)batch * hs, 0);
  AL(au.items, au.items_cap, 0);
  AL(au.n_states, batch, 0);
  au.st_stride = (g->dev.T + 63u) & ~63u;
  AL(au.st, (size_t)batch * au.st_stride, 0xFF);
  au.req_cap = 1u << 20;
  AL(au.req, au.req_cap, 0);
  AL(au.job_info, batch, 0);
  AL(rt.n_roots, 4, 0);
  AL(rt.tops, TOP_N, 0);
  AL(rt.counters, CNT_TOTAL, 0);
  if (rt.on) {  // the cache of context-independent entries and the frames of the rows' sweeps
    AL(rt.hash, rh, 0);
    AL(rt.info, (size_t)rt.max_roots * RI_WORDS, 0);
    AL(rt.charts, rt.charts_cap, 0);
    AL(rt.ci_rows, (size_t)rt.max_roots * g->dev.Wm, 0);
    AL(rt.states, rt.st_cap, 0);
    AL(rt.items, rt.it_cap, 0);
    AL(rt.trans, rt.tr_cap, 0);
    AL(rt.pending, rt.pend_cap, 0);
    AL(rt.rj_chart, batch, 0);
    AL(rt.rj_mask, batch, 0);
    AL(rt.rj_flags, batch, 0);
    AL(rt.rj_jobs, batch, 0);
    AL(d.cx.bind, (size_t)batch * rt.max_ph, 0);
    AL(d.cx.jobs, batch, 0);
    AL(d.cx.ctab, (size_t)batch * CT_SLOTS, 0);
    AL(d.cx.fjobs, batch, 0);
    AL(d.cx.frames, (size_t)batch * MAXF, 0);
    AL(d.cx.fbind, (size_t)batch * MAXF * rt.max_ph, 0);
    AL(d.cx.frame_ctr, batch, 0);
    AL(d.cx.st32, (size_t)batch * au.st_stride, 0xFF);
    d.cx.req2_cap = 1u << 20;
    AL(d.cx.req2, d.cx.req2_cap, 0);
  }
  AL(s->init_state_dev, 4, 0xFF);
  AL(s->result_dev, 4, 0);
  AL(s->query_dev, (size_t)batch * 16, 0);
#undef AL
  if (e != cudaSuccess) {
    fmt_status stt = cuda_fail(e, "allocating the sequence state");
    delete s;
    return stt;
  }
  if (d.cache_on && !(opt && opt->cache_keep_when_full)) {
    void* dp = nullptr;
    if (cudaHostAlloc((void**)&s->full_flag_host, sizeof(uint32_t), cudaHostAllocMapped) == cudaSuccess &&
        cudaHostGetDevicePointer(&dp, s->full_flag_host, 0) == cudaSuccess) {
      *s->full_flag_host = 0u;
      d.full_flag = static_cast<uint32_t*>(dp);
    } else {  // no mapped memory: the cache simply stops taking entries when it is full
      if (s->full_flag_host) cudaFreeHost(s->full_flag_host);
      s->full_flag_host = nullptr;
      cudaGetLastError();
    }
  }
  launch_init(g->dev, d, s->result_dev, st);
  launch_intern_init(d, s->init_state_dev, st);
  launch_reset(d, nullptr, batch, s->init_state_dev, st);
  int32_t result = 0;
  e = cudaMemcpyAsync(&result, s->result_dev, 4, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) {
    fmt_status stt = cuda_fail(e, "building the start chart");
    delete s;
    return stt;
  }
  if (result != 1) {
    delete s;
    return fail(FMT_ERR_CAPACITY, "the start chart does not fit the configured capacities");
  }
  s->device_bytes = s->bufs.bytes;
  *out = s;
  return FMT_OK;
}

void fmt_state_destroy(fmt_state* s) { delete s; }

static fmt_status launched(const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, what);
  return FMT_OK;
}

fmt_status fmt_state_reset(fmt_state* s, const uint32_t* rows_dev, uint32_t n, void* stream) {
  if (!s) return fail(FMT_ERR_INVALID_ARG, "NULL state");
  if (!rows_dev && n > s->dev.B) return fail(FMT_ERR_INVALID_ARG, "n exceeds the batch");
  launch_reset(s->dev, rows_dev, n, s->init_state_dev, (cudaStream_t)stream);
  return launched("fmt_state_reset");
}

static fmt_status cache_turn_over(fmt_state* s, cudaStream_t st);

fmt_status fmt_state_advance(fmt_state* s, const int32_t* token_ids_dev, int32_t* status_dev, void* stream) {
  if (!s || !token_ids_dev) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  if (s->full_flag_host) {
    volatile uint32_t* flag = s->full_flag_host;
    if (s->skip_full_check) {  // kernels enqueued before the last flush may have raised the flag once more
      *flag = 0u;
      s->skip_full_check = false;
    } else if (*flag) {
      *flag = 0u;
      s->skip_full_check = true;
      ++s->flushes;
      if (fmt_status rc = cache_turn_over(s, (cudaStream_t)stream)) return rc;
    }
  }
  cudaEvent_t e0, e1;
  s->prof.next(0, &e0, &e1);
  if (e0) cudaEventRecord(e0, (cudaStream_t)stream);
  launch_advance(s->g->dev, s->dev, token_ids_dev, status_dev, (cudaStream_t)stream);
  if (e1) cudaEventRecord(e1, (cudaStream_t)stream);
  return launched("fmt_state_advance");
}

fmt_status fmt_state_forced_bytes(fmt_state* s, uint8_t* bytes_dev, size_t stride_bytes, uint32_t* len_dev, uint32_t max_len,
                                  void* stream) {
  if (!s || !bytes_dev || !len_dev) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  if (max_len > FMT_MAX_FORCED_BYTES) max_len = FMT_MAX_FORCED_BYTES;
  if (stride_bytes < max_len) return fail(FMT_ERR_INVALID_ARG, "stride_bytes is smaller than max_len");
  launch_forced(s->g->dev, s->dev, bytes_dev, stride_bytes, len_dev, max_len, (cudaStream_t)stream);
  return launched("fmt_state_forced_bytes");
}

fmt_status fmt_fill_mask(fmt_state* s, uint32_t* mask_dev, size_t stride_words, void* stream) {
  if (!s || !mask_dev) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  if (stride_words < s->g->dev.Wm) return fail(FMT_ERR_INVALID_ARG, "stride_words is smaller than ceil(V/32)");
  cudaStream_t st = (cudaStream_t)stream;
  cudaEvent_t w0, w1, r0 = nullptr, r1 = nullptr;
  if (s->dev.rt.on) s->prof.next(3, &r0, &r1);
  s->prof.next(1, &w0, &w1);
  if (cudaError_t e = next_generations(s, st)) return cuda_fail(e, "fmt_fill_mask");
  launch_fill(s->g->dev, s->dev, s->sweep_grid, st, r0, r1, w0, w1);
  launch_gather(s->g->dev, s->dev, mask_dev, stride_words, st);
  return launched("fmt_fill_mask");
}

fmt_status fmt_apply_mask(const uint32_t* mask_dev, size_t stride_words, void* logits_dev, fmt_dtype dtype,
                          uint32_t batch, uint32_t V, size_t row_stride_elems, void* stream) {
  if (!mask_dev || !logits_dev) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  if (dtype != FMT_BF16 && dtype != FMT_FP32) return fail(FMT_ERR_INVALID_ARG, "unknown dtype");
  if (stride_words < (V + 31) / 32 || row_stride_elems < V) return fail(FMT_ERR_INVALID_ARG, "a stride is too small");
  if (batch > 65535) return fail(FMT_ERR_INVALID_ARG, "batch above 65535");
  launch_apply(mask_dev, stride_words, logits_dev, (int)dtype, batch, V, row_stride_elems, (cudaStream_t)stream);
  return launched("fmt_apply_mask");
}

fmt_status fmt_fill_and_apply(fmt_state* s, uint32_t* mask_dev_or_null, size_t stride_words, void* logits_dev,
                              fmt_dtype dtype, size_t row_stride_elems, void* stream) {
  if (!s || !logits_dev) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  if (dtype != FMT_BF16 && dtype != FMT_FP32) return fail(FMT_ERR_INVALID_ARG, "unknown dtype");
  if (mask_dev_or_null && stride_words < s->g->dev.Wm)
    return fail(FMT_ERR_INVALID_ARG, "stride_words is smaller than ceil(V/32)");
  if (row_stride_elems < s->g->dev.V) return fail(FMT_ERR_INVALID_ARG, "row_stride_elems is smaller than V");
  cudaStream_t st = (cudaStream_t)stream;
  cudaEvent_t w0, w1, a0, a1, r0 = nullptr, r1 = nullptr;
  if (s->dev.rt.on) s->prof.next(3, &r0, &r1);
  s->prof.next(1, &w0, &w1);
  s->prof.next(2, &a0, &a1);
  if (cudaError_t e = next_generations(s, st)) return cuda_fail(e, "fmt_fill_and_apply");
  launch_fill(s->g->dev, s->dev, s->sweep_grid, st, r0, r1, w0, w1);
  if (a0) cudaEventRecord(a0, st);
  launch_gather_apply(s->g->dev, s->dev, logits_dev, (int)dtype, row_stride_elems, mask_dev_or_null, stride_words, st);
  if (a1) cudaEventRecord(a1, st);
  return launched("fmt_fill_and_apply");
}

fmt_status fmt_state_cache_clear(fmt_state* s, void* stream) {
  if (!s) return fail(FMT_ERR_INVALID_ARG, "NULL state");
  if (!s->dev.cache_on) return FMT_OK;
  cudaStream_t st = (cudaStream_t)stream;
  StateDev& d = s->dev;
  launch_evacuate(d, st);
  cudaError_t e = cudaMemsetAsync(d.ht, 0, ((size_t)d.ht_mask + 1) * 4, st);
  // the cache ids are handed out anew: what was learnt about (id, token) pairs goes too
  if (e == cudaSuccess) e = cudaMemsetAsync(d.tr_key, 0, ((size_t)d.tr_mask + 1) * 8, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(d.tr_val, 0x80, ((size_t)d.tr_mask + 1) * 4, st);
  // counters: states, mask rows, jobs, work, error flag, pool top
  if (e == cudaSuccess) e = cudaMemsetAsync(d.counters, 0, 8 * 4, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(d.st_ref, 0, d.max_states, st);
  if (e != cudaSuccess) return cuda_fail(e, "fmt_state_cache_clear");
  launch_reintern(d, s->init_state_dev, st);
  return launched("fmt_state_cache_clear");
}

// The cache has no room left: switch to the other generation of its storage, enter the rows' current charts
// again and carry over every entry that was found again after it was made, with its mask row.
static fmt_status cache_turn_over(fmt_state* s, cudaStream_t st) {
  if (!s->st_off2[1]) return fmt_state_cache_clear(s, st);
  const StateDev old = s->dev;
  StateDev& d = s->dev;
  launch_evacuate(old, st);  // rows whose chart lives in the cache's storage take it along
  cudaError_t e = cudaMemcpyAsync(s->old_count_dev, old.counters + CNT_N_STATES, 4, cudaMemcpyDeviceToDevice, st);
  s->generation ^= 1;
  const int gi = s->generation;
  d.st_off = s->st_off2[gi], d.st_mask = s->st_mask2[gi], d.st_ref = s->st_ref2[gi];
  d.pool_base = s->pool_base2[gi];
  d.mrow_base = s->mrow_base2[gi];
  if (e == cudaSuccess) e = cudaMemsetAsync(d.ht, 0, ((size_t)d.ht_mask + 1) * 4, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(d.tr_key, 0, ((size_t)d.tr_mask + 1) * 8, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(d.tr_val, 0x80, ((size_t)d.tr_mask + 1) * 4, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(d.counters, 0, 8 * 4, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(d.st_ref, 0, d.max_states, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(d.st_mask, 0xFF, (size_t)d.max_states * 4, st);
  if (e != cudaSuccess) return cuda_fail(e, "emptying the state cache");
  launch_reintern(d, s->init_state_dev, st);
  launch_survivors(s->g->dev, old, d, s->old_count_dev, st);
  return launched("emptying the state cache");
}

fmt_status fmt_state_ci_cache_clear(fmt_state* s, void* stream) {
  if (!s) return fail(FMT_ERR_INVALID_ARG, "NULL state");
  cudaStream_t st = (cudaStream_t)stream;
  RootDev& r = s->dev.rt;
  if (!r.on) return FMT_OK;  // (the state was created without that cache)
  cudaError_t e = cudaMemsetAsync(r.hash, 0, ((size_t)r.hash_mask + 1) * 4, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(r.n_roots, 0, 4, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(r.tops, 0, TOP_N * 4, st);

  if (e != cudaSuccess) return cuda_fail(e, "fmt_state_ci_cache_clear");
  return FMT_OK;
}

fmt_status fmt_state_set_wait_limit(fmt_state* s, uint32_t log2_polls) {
  if (!s) return fail(FMT_ERR_INVALID_ARG, "NULL state");
  s->dev.poll_limit_shift = std::min(log2_polls, 30u);
  return FMT_OK;
}

fmt_status fmt_state_query(fmt_state* s, uint8_t* accepting, uint8_t* finished, uint32_t* n_sets, uint32_t* n_items,
                           int32_t* state_id, void* stream) {
  if (!s) return fail(FMT_ERR_INVALID_ARG, "NULL state");
  cudaStream_t st = (cudaStream_t)stream;
  const uint32_t B = s->dev.B;
  uint8_t* q = s->query_dev;
  uint8_t* a = q;
  uint8_t* f = q + B;
  uint32_t* ns = reinterpret_cast<uint32_t*>(q + 4 * (size_t)B);
  uint32_t* ni = ns + B;
  int32_t* sid = reinterpret_cast<int32_t*>(ni + B);
  launch_query(s->dev, a, f, ns, ni, sid, st);
  std::vector<uint8_t> host((size_t)B * 16);
  cudaError_t e = cudaMemcpyAsync(host.data(), q, host.size(), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e, "fmt_state_query");
  if (accepting) memcpy(accepting, host.data(), B);
  if (finished) memcpy(finished, host.data() + B, B);
  if (n_sets) memcpy(n_sets, host.data() + 4 * (size_t)B, 4 * (size_t)B);
  if (n_items) memcpy(n_items, host.data() + 8 * (size_t)B, 4 * (size_t)B);
  if (state_id) memcpy(state_id, host.data() + 12 * (size_t)B, 4 * (size_t)B);
  return FMT_OK;
}

fmt_status fmt_state_copy_chart(fmt_state* s, uint32_t row, uint32_t* out, size_t cap_words, size_t* n_words,
                                void* stream) {
  if (!s || !n_words || row >= s->dev.B) return fail(FMT_ERR_INVALID_ARG, "bad argument");
  cudaStream_t st = (cudaStream_t)stream;
  uint64_t off = 0;
  cudaError_t e = cudaMemcpyAsync(&off, s->dev.row_chart + row, 8, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  uint32_t hdr[CH_HDR];
  if (e == cudaSuccess) e = cudaMemcpyAsync(hdr, s->dev.arena + off, sizeof(hdr), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e, "fmt_state_copy_chart");
  *n_words = hdr[CH_WORDS];
  size_t n = std::min<size_t>(cap_words, hdr[CH_WORDS]);
  if (out && n) {
    e = cudaMemcpyAsync(out, s->dev.arena + off, n * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "fmt_state_copy_chart");
  }
  return FMT_OK;
}

fmt_status fmt_state_set_profiling(fmt_state* s, int enable) {
  if (!s) return fail(FMT_ERR_INVALID_ARG, "NULL state");
  s->prof.on = (enable & 1) != 0;
  s->dev.time_steps = (enable & 2) ? 1u : 0u;
  return FMT_OK;
}

fmt_status fmt_state_read_profile_series(fmt_state* s, int kind, float* ms_out, size_t cap, size_t* n) {
  if (!s || !n || kind < 0 || kind > 3) return fail(FMT_ERR_INVALID_ARG, "bad argument");
  *n = s->prof.used[kind];
  for (size_t i = 0; i < s->prof.used[kind] && i < cap && ms_out; ++i) {
    cudaError_t e = cudaEventSynchronize(s->prof.b[kind][i]);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms_out[i], s->prof.a[kind][i], s->prof.b[kind][i]);
    if (e != cudaSuccess) return cuda_fail(e, "fmt_state_read_profile_series");
  }
  return FMT_OK;
}

fmt_status fmt_state_read_profile(fmt_state* s, fmt_profile* out) {
  if (!s || !out) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  double ms[4] = {0, 0, 0, 0};
  for (int k = 0; k < 4; ++k) {
    for (size_t i = 0; i < s->prof.used[k]; ++i) {
      cudaError_t e = cudaEventSynchronize(s->prof.b[k][i]);
      float t = 0.f;
      if (e == cudaSuccess) e = cudaEventElapsedTime(&t, s->prof.a[k][i], s->prof.b[k][i]);
      if (e != cudaSuccess) return cuda_fail(e, "fmt_state_read_profile");
      ms[k] += t;
    }
  }
  out->advance_ms = ms[0], out->sweep_ms = ms[1], out->apply_ms = ms[2];
  out->advance_launches = s->prof.used[0], out->sweep_launches = s->prof.used[1], out->apply_launches = s->prof.used[2];
  out->roots_ms = ms[3], out->roots_launches = s->prof.used[3];
  s->prof.used[0] = s->prof.used[1] = s->prof.used[2] = s->prof.used[3] = 0;
  return FMT_OK;
}

fmt_status fmt_state_copy_counters(fmt_state* s, int which, uint32_t* out, size_t cap_words, size_t* n_words, void* stream) {
  if (!s || !n_words || which < 0 || which > 1) return fail(FMT_ERR_INVALID_ARG, "bad argument");
  *n_words = CNT_TOTAL;
  const size_t n = std::min<size_t>(cap_words, CNT_TOTAL);
  if (out && n) {
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(out, which ? s->dev.rt.counters : s->dev.counters, n * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "fmt_state_copy_counters");
  }
  return FMT_OK;
}

fmt_status fmt_get_stats(fmt_state* s, fmt_stats* out, void* stream) {
  if (!s || !out) return fail(FMT_ERR_INVALID_ARG, "NULL argument");
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t c[CNT_TOTAL];
  cudaError_t e = cudaMemcpyAsync(c, s->dev.counters, sizeof(c), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e, "fmt_get_stats");
  auto u64 = [&](uint32_t slot) { return (uint64_t)c[slot] | ((uint64_t)c[slot + 1] << 32); };
  out->steps_advanced = u64(CNT_STAT_ADV);
  out->fills = u64(CNT_STAT_FILLS);
  out->fills_computed = u64(CNT_STAT_COMPUTED);
  out->fills_from_cache = u64(CNT_STAT_CACHED);
  out->fills_shared = u64(CNT_STAT_SHARED);
  out->states_cached = std::min<uint64_t>(c[CNT_N_STATES], s->dev.max_states);
  out->mask_rows_cached = std::min<uint64_t>(c[CNT_N_MASK_ROWS], s->dev.max_mask_rows);
  out->pool_words_used = std::min<uint64_t>(u64(CNT_POOL_LO), s->dev.pool_words);
  out->chart_items_max = c[CNT_STAT_ITEMS_MAX];
  out->chart_sets_max = c[CNT_STAT_SETS_MAX];
  out->capacity_errors = u64(CNT_STAT_CAPERR);
  out->big_mode_units = u64(CNT_STAT_BIG);
  out->sweep_transitions = u64(CNT_STAT_TRANS);
  out->sweep_states = u64(CNT_STAT_LOCAL);
  out->advances_cached = u64(CNT_STAT_ADV_HIT);
  out->rows_from_root = u64(CNT_STAT_JOBS_ROOT);
  out->rows_plain = s->dev.rt.on ? u64(CNT_STAT_JOBS_PLAIN) : u64(CNT_STAT_COMPUTED);  // (without that cache every computed row is swept from its chart)
  // (rows swept from their chart's last set without frames count their steps in the sweep's own slots)
  out->walk_transitions = u64(CNT_STAT_CTX_TRANS) + u64(CNT_STAT_TRANS);
  out->walk_states = u64(CNT_STAT_CTX_STATES) + u64(CNT_STAT_LOCAL);
  out->rows_mask_only = u64(CNT_STAT_JOBS_MASK);
  out->walk_frames = u64(CNT_STAT_FRAMES);
  out->root_sweeps = u64(CNT_STAT_ROOT_SWEEPS);
  out->fills_aborted = u64(CNT_STAT_ABORTS);
  out->device_bytes = s->device_bytes;
  out->cache_flushes = s->flushes;
  out->earley_step_cycles = u64(CNT_STAT_STEP_CYCLES);
  out->advance_chart_words = u64(CNT_STAT_ADV_WORDS);
  for (int i = 0; i < 8; ++i) out->diag[i] = c[CNT_DIAG + i];
  // the root sweeps count their Earley steps in counters of their own
  uint32_t n_roots = 0;
  e = cudaMemcpyAsync(c, s->dev.rt.counters, sizeof(c), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(&n_roots, s->dev.rt.n_roots, 4, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e, "fmt_get_stats");
  out->sweep_transitions = u64(CNT_STAT_TRANS);
  out->sweep_states = u64(CNT_STAT_LOCAL);
  out->big_mode_units += u64(CNT_STAT_BIG);
  out->earley_step_cycles += u64(CNT_STAT_STEP_CYCLES);
  for (int i = 0; i < 8; ++i) out->diag[8 + i] = c[CNT_DIAG + i];
  out->roots = std::min<uint64_t>(n_roots, s->dev.rt.max_roots);
  return FMT_OK;
}

}  // extern "C"
