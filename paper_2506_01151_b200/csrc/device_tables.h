// Device-side views of the compiled grammar / vocabulary and of a batch of sequences.
#pragma once
#include <cstdint>

namespace fmt {

struct GrammarDev {
  uint32_t D, N, C, Nw;          // dotted rules, non-terminals, byte classes, words per non-terminal bitset
  uint32_t V, Wm, T, depth;      // vocabulary, mask words, trie nodes, longest token
  int32_t eos;
  uint32_t start_nullable;
  const uint32_t* info;          // [D]
  const uint16_t* lhs;           // [D]
  const uint32_t* class_bits;    // [C][8]
  const uint8_t* eq_of_byte;     // [256] equivalence class of each byte (same membership in all byte classes)
  uint32_t n_eq;
  const uint32_t* nt_closure;    // [N][Nw]
  const uint32_t* direct_off;    // [N+1]
  const uint16_t* direct_items;
  const uint8_t* node_byte;      // [T]
  const uint32_t* parent;        // [T]
  const uint8_t* node_depth;     // [T]
  // The tables above that every Earley step reads (info, class_bits, eq_of_byte, nt_closure,
  // direct_off, direct_items) sit in one contiguous block so that a kernel can copy them into
  // shared memory at once and shift the six pointers.
  const uint32_t* hot_block;
  uint32_t hot_words;
  const uint32_t* lvl_off;       // [depth+2]
  const uint32_t* tok_node;      // [V]
  const uint32_t* vocab_off;     // [V+1]
  const uint8_t* vocab_bytes;
};

// A pruned chart in memory (uint32 words):
//   [0] number of live Earley sets m      [1] total items          [2] flags (bit 0: accepting)
//   [3] hash low   [4] hash high          [5] total words          [6],[7] unused
//   [8 .. 8+m]     set_off[m+1]: first item of each set
//   then the items, (origin << 16) | dotted-rule id, ascending within each set; origins index
//   the live sets 0..m-1 (the dense renumbering that makes equal situations equal charts).
constexpr uint32_t CH_SETS = 0, CH_ITEMS = 1, CH_FLAGS = 2, CH_HASH_LO = 3, CH_HASH_HI = 4, CH_WORDS = 5, CH_HDR = 8;
constexpr uint32_t CHART_ACCEPTING = 1u;

constexpr uint32_t ROW_FINISHED = 1u, ROW_BROKEN = 2u;

// counters[] slots
enum : uint32_t {
  CNT_N_STATES = 0,
  CNT_N_MASK_ROWS = 1,
  CNT_N_JOBS = 2,
  CNT_ERR = 4,          // sticky: some device routine hit a capacity limit
  CNT_AUTO_ITEMS = 5,   // top of the automaton's item pool (words), reset by every fill
  CNT_POOL_LO = 6,      // 64-bit pool top (words) lives in slots 6,7 (8-byte aligned)
  CNT_STAT_ADV = 8,     // 64-bit statistics from here on, two slots each
  CNT_STAT_FILLS = 10,
  CNT_STAT_COMPUTED = 12,
  CNT_STAT_CACHED = 14,
  CNT_STAT_SHARED = 16,
  CNT_STAT_ITEMS_MAX = 18,
  CNT_STAT_SETS_MAX = 20,
  CNT_STAT_CAPERR = 22,
  CNT_STAT_BIG = 24,
  CNT_STAT_TRANS = 26,  // transitions computed by the trie sweep (Earley steps)
  CNT_STAT_LOCAL = 28,  // local states created by the trie sweep
  CNT_BAR = 30,         // grid barrier of the trie sweep: arrivals
  CNT_BAR_ERR = 31,     // a block gave up waiting at the barrier
  CNT_LEVEL_ALIVE = 32, // [MAX_TOKEN_BYTES + 2] per trie depth: some node of some job was alive
  CNT_LEVEL_REQ = 68,   // [MAX_TOKEN_BYTES + 2] per trie depth: transitions queued for computation
  CNT_HASH_GEN = 104,   // generation of the sweep's per-job hashes (1 .. 65535), advanced by every fill
  CNT_HASH_CLEAR = 105, // this fill starts the generations over: the sweep clears the hashes first
  CNT_STAT_ADV_HIT = 106,  // 64-bit: advances answered by the transition cache
  CNT_LEVEL_TAKEN = 108,   // [MAX_TOKEN_BYTES + 2] per trie depth: tickets drawn for the queued transitions
  CNT_PASS_DONE = 144,     // CTAs that have finished their part of a depth's pass (summed over the depths)
  CNT_TOTAL = 146
};

// Per-job automaton of hash-consed Earley sets, built on demand by the trie walk.  A "local
// state" is the Earley set reached from the job's base chart by some byte string; equal sets get
// one id, so a transition (state, byte class) is computed once per job, whatever the number of
// trie nodes that need it.  Items of a local state name their origin as: a set index of the base
// chart (< m), m + k for local state k, or ORIGIN_SELF for the state itself.
// Record of a state (rec_words uint32, a multiple of 32, so records never share a 128-byte line):
//   [0] first item (word offset into items)  [1] item count  [2] hash of the kernel  [3] items of the
//   kernel (they come first)  [4..11] scannable bytes
//   [16 .. 16+n_eq) transition per byte class: T_UNKNOWN, T_PENDING (a warp is computing it),
//                   T_DEAD or the next state's id
struct AutoDev {
  uint32_t cap;        // states per job, state 0 being the base chart's last set
  uint32_t rec_words;
  uint32_t hash_mask;  // hash slots per job - 1
  uint32_t items_cap;  // words of the item pool shared by all jobs
  uint32_t* recs;      // [jobs][cap][rec_words]
  uint32_t* hash;      // [jobs][hash_mask + 1], id + 1 or 0
  uint32_t* items;     // [items_cap]
  uint32_t* n_states;  // [jobs]
  uint16_t* st;        // [jobs][st_stride] local state reached at every trie node (ST_DEAD if none)
  uint32_t st_stride;
  unsigned long long* req;  // [req_cap] transitions to compute at the current depth: job << 32 | state << 8 | byte
  uint32_t req_cap;
  uint32_t smem_bytes;      // dynamic shared memory of the sweep kernel
  uint32_t tables_in_smem;  // 1: the grammar's hot tables are staged in shared memory
  uint4* job_info;          // [jobs] x: chart offset low, y: chart offset high, z: live sets m, w: row | accepting << 31
};
constexpr uint16_t ST_DEAD = 0xFFFFu, ST_PENDING = 0xFFFEu;
constexpr uint32_t T_UNKNOWN = 0xffffffffu, T_DEAD = 0xfffffffeu, T_FAIL = 0xfffffffdu, T_PENDING = 0xfffffffcu;
constexpr uint32_t ORIGIN_SELF = 0xFFFFu;
constexpr uint32_t AR_ITEMS = 0, AR_N = 1, AR_HASH = 2, AR_NK = 3, AR_SCAN = 4, AR_TRANS = 16;

struct StateDev {
  uint32_t B;
  uint32_t chart_words;       // capacity of one private chart buffer
  uint32_t cache_on;
  uint32_t max_states, ht_mask, max_mask_rows;
  uint64_t pool_base, pool_words;   // word offsets into arena / size of the pool
  uint64_t init_off;                // word offset of the start chart
  uint32_t* arena;            // [B*3 private buffers][start chart][pool]
  uint64_t* row_chart;        // [B] word offset of the row's current chart
  uint8_t* row_buf;           // [B] private buffer holding it (0..2) or 255 (pool / start chart)
  int32_t* row_state;         // [B] cache id or -1
  uint32_t* row_flags;        // [B]
  int32_t* row_mask;          // [B] mask row holding the row's mask after a fill (or a special value)
  uint32_t* ht;               // [ht_mask+1] id+1, 0 = empty
  uint64_t* st_off;           // [max_states] word offset of the cached chart
  int32_t* st_mask;           // [max_states] -1 none, >= 0 mask row, <= -2 claimed by row -(x+2)
  uint32_t* mask_rows;        // [B + max_mask_rows][Wm]; rows 0..B-1 are per-row scratch
  // transition cache of advance: (cache id of a chart, token) -> cache id of the next chart, or TR_REJECT.
  // Open addressing; tr_key holds (id + 1) << 32 | token, 0 = empty; tr_val is TR_UNSET until the value is there.
  unsigned long long* tr_key; // [tr_mask + 1]
  int32_t* tr_val;            // [tr_mask + 1]
  uint32_t tr_mask;
  uint32_t* jobs;             // [B] rows whose mask must be computed
  uint32_t* counters;         // [CNT_TOTAL]
  uint32_t* big_scratch;      // per-warp large scratch areas of the trie walk
  uint32_t big_arena_items, big_hset_slots;
  AutoDev au;
};

constexpr int32_t TR_REJECT = -2;                 // tr_val: the token cannot follow
constexpr int32_t TR_UNSET = (int32_t)0x80808080;  // tr_val: not written yet (the arrays are filled with byte 0x80)
constexpr int32_t MASK_ZERO = -1;       // row_mask: all-zero mask (broken row)
constexpr int32_t MASK_EOS_ONLY = -2;   // row_mask: finished row
constexpr int32_t MASK_ALIAS0 = -10;    // row_mask <= MASK_ALIAS0: same mask as row (MASK_ALIAS0 - x)

}  // namespace fmt
