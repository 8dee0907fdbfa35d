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
  // regular non-terminals run as automata: item id dfa_first + g is automaton state g
  uint32_t dfa_first;
  const uint16_t* dfa_trans;     // [states][n_eq] target | 0x4000 target has transitions | 0x8000 target accepts, or 0xFFFF
  const uint16_t* dfa_done;      // [states] completed item of the state's non-terminal
  const uint32_t* dfa_scan;      // [states][8] bytes with a transition
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
  const uint32_t* child_off;     // [T+1] children of node n are nodes child_off[n] .. child_off[n+1]-1
  const uint32_t* tok_off;       // [T+1] tokens whose bytes end at node n (duplicates included)
  const uint32_t* tok_ids;
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
  CNT_N_FJOBS = 3,      // jobs that go through the level sweep of the fill
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
  CNT_HASH_GEN = 104,   // (the depth counters that every fill clears end here; the fills' generations are handed out by the host)
  CNT_STAT_ADV_HIT = 106,  // 64-bit: advances answered by the transition cache
  CNT_LEVEL_TAKEN = 108,   // [MAX_TOKEN_BYTES + 2] per trie depth: tickets drawn for the queued transitions
  CNT_PASS_DONE = 144,     // CTAs that have finished their part of a depth's pass (summed over the depths)
  CNT_LAST_LEVEL = 145,    // deepest trie depth the last sweep visited
  CNT_STAT_CTX_TRANS = 146,    // 64-bit: Earley steps of the context-dependent walk
  CNT_STAT_CTX_STATES = 148,   // 64-bit: Earley sets it created
  CNT_STAT_ROOT_SWEEPS = 150,  // 64-bit: roots whose context-independent part was swept
  CNT_STAT_JOBS_ROOT = 152,    // 64-bit: computed rows that started from a swept root
  CNT_STAT_JOBS_PLAIN = 154,   // 64-bit: computed rows that walked the whole trie themselves
  CNT_STAT_JOBS_MASK = 156,    // 64-bit: computed rows answered by their root's mask row alone
  CNT_STAT_ABORTS = 160,       // 64-bit: fills abandoned because a bounded wait ran out
  CNT_STAT_STEP_CYCLES = 162,  // 64-bit: SM cycles spent inside Earley steps of the fill (summed over warps)
  CNT_STAT_ADV_WORDS = 164,    // 64-bit: chart words read and written by advance
  CNT_STAT_FRAMES = 184,       // 64-bit: frames made (sets of a walk recognised as roots)
  CNT_DIAG = 166,              // [16] where capacity errors and expired waits came from (see DIAG_*)
  CNT_TOTAL = 186
};

enum : uint32_t {
  DIAG_SET_TABLE = 0,    // a job's table of Earley sets is full
  DIAG_ITEM_POOL = 1,    // the fill's item pool is full
  DIAG_SET_SCRATCH = 2,  // a set outgrew even the large per-warp scratch
  DIAG_QUEUE_FULL = 3,   // the walk's queue (or a depth's queue of the sweep) is full
  DIAG_WAIT_VALUE = 4,   // a wait for a transition another warp was computing ran out
  DIAG_WAIT_QUEUE = 5,   // a wait for queued work ran out
  DIAG_WAIT_GRID = 6,    // a wait for the other thread blocks ran out
  DIAG_ROOT_FAILED = 7,  // a root's sweep could not be kept
  DIAG_N = 16
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
constexpr uint32_t T_CTX = 0xfffffffau;  // the transition needs the sequence's own chart (context-dependent)
constexpr uint16_t ST_CTX = 0xFFFDu;
constexpr uint32_t ORIGIN_SELF = 0xFFFFu;
constexpr uint32_t AR_ITEMS = 0, AR_N = 1, AR_HASH = 2, AR_NK = 3, AR_SCAN = 4, AR_TRANS = 16;

// ---- Context-independent part of a mask, computed once per "root" (Section 4.3).
// A root is the last Earley set of a chart with its origins made anonymous: the k distinct origins
// of its scanned / completed items become placeholders 0..k-1 (ascending), the set's own index
// becomes k.  The trie sweep over the root's one-set chart, in which a completion that would have
// to read a placeholder set answers T_CTX instead, yields
//   - the tokens valid whatever the rest of the chart holds (one mask row per root) and the number of
//     trie nodes at which the chart would have been needed (none: the row is the whole answer),
//   - the Earley sets met on the way (the root's "region": their items, which an Earley step of a
//     sequence reads with the placeholders bound to its chart's set indices) and the transitions
//     between them, one 16-bit entry per (set, byte class).
// Origin codes inside a sequence's walk: [0, LBASE) a set of its chart, [LBASE, RBASE) a set the
// walk made, [RBASE, ORIGIN_SELF) set (code - RBASE) of the root's region (0 = the root set).
constexpr uint32_t LBASE = 0x800u, RBASE = 0x8000u;
constexpr uint32_t ROOT_NONE = 0xffffffffu;
enum : uint32_t { ROOT_NEW = 0, ROOT_READY = 1, ROOT_FAILED = 2 };
enum : uint32_t {  // words of a root's directory entry
  RI_STATUS = 0, RI_P = 1, RI_NK = 2, RI_N = 3, RI_HASH = 4, RI_CHART = 5, RI_FR_N = 7,
  RI_ST_OFF = 8, RI_NSTATES = 9, RI_TR_OFF = 10, RI_WORDS = 16
};
enum : uint32_t { TOP_CHARTS = 0, TOP_STATES = 2, TOP_ITEMS = 3, TOP_TRANS = 4, TOP_PENDING = 7, TOP_N = 8 };
constexpr uint16_t R_DEAD = 0xFFFFu, R_CTX = 0xFFFEu;  // values of a region's transition table besides set numbers

struct RootDev {
  uint32_t on;           // 0: every computed row walks the whole trie itself
  uint32_t max_roots, hash_mask;
  uint32_t max_items;    // a last set with more items than this is not made a root
  uint32_t max_ph;       // nor one with more distinct origins than this
  uint32_t* hash;        // [hash_mask + 1] root id + 1, 0 = empty
  uint32_t* info;        // [max_roots][RI_WORDS]
  uint32_t* n_roots;
  uint32_t* charts;      // pool of one-set charts, the key of a root (the scanned / completed items come first)
  uint32_t charts_cap;
  uint32_t* ci_rows;     // [max_roots][Wm]
  uint2* states;         // pool: per region set x = first item (in `items`), y = item count
  uint32_t st_cap;
  uint32_t* items;       // pool
  uint32_t it_cap;
  uint16_t* trans;       // pool: per region set one entry per byte class: the set reached, R_DEAD or R_CTX
  uint32_t tr_cap;
  uint32_t* tops;        // [TOP_N] tops of the pools
  // roots made by a walk (a set it met had no entry yet): swept by the next fill
  uint32_t* pending;         // [pend_cap] root ids
  uint32_t pend_cap;
  uint32_t* counters;    // [CNT_TOTAL] counters of the root sweep (its own barrier, queue and job counts)
  // the roots to sweep in this fill, as the rows of the sweep's view of the state
  uint64_t* rj_chart;    // [B] word offset of the root's chart in `charts`
  int32_t* rj_mask;      // [B] root id = its row in ci_rows
  uint32_t* rj_flags;    // [B]
  uint32_t* rj_jobs;     // [B] identity
};

// What the context-dependent walk needs to know about a job (a row whose mask is computed).
struct CtxJob {
  uint64_t chart_off;    // the row's chart (word offset into the arena)
  uint32_t m;            // its live sets
  uint32_t row_acc;      // row | accepting << 31
  uint32_t root;         // root id or ROOT_NONE (the walk starts at the trie's first level from the chart's last set)
  uint32_t P;            // placeholders of the root
  uint32_t spare[3];
  int32_t mrow;          // mask row to write
  uint32_t pad[2];
};

// A frame: a root's region as one job sees it, with the root's placeholders bound to sets of the job's
// chart.  Frame 0 is the job's own root; further frames appear when a context-dependent step of the
// walk lands on a set that is itself a known root (what follows it is context-independent again).
// Set k of a frame is named by the code RBASE + k, in every frame: which frame is meant follows from
// where the code stands.  A set made by a step out of a frame's set lives "in" that frame (the frame
// codes among its origins mean that frame's sets), and so does every set made from it; a set whose
// origins all lie in the chart depends on no frame, and only such a set can open a frame of its own.
struct Frame {
  uint32_t root, P, n, st_off, tr_off, pad0, pad1, pad2;
};
constexpr uint32_t MAXF = 255;        // frames per job
constexpr uint32_t NOFRAME = 0xffffffffu;
constexpr uint32_t AR_FRAME = 12;     // word of a walk's set record: 0 not looked up yet, NOFRAME, or frame + 1 (the frame it opens)
constexpr uint32_t AR_SALT = 13;      // word of a set record: 0, or frame + 1 (the frame the set lives in)

constexpr uint32_t CT_SLOTS = 4096;  // per job: remembered transitions out of region sets (power of two)

struct CtxDev {
  uint16_t* bind;              // [B][max_ph] the chart set each placeholder stands for
  CtxJob* jobs;                // [B]
  unsigned long long* ctab;    // [B][CT_SLOTS] generation << 48 | (frame + 1) << 40 | set code << 24 | byte class << 16 | value
  uint32_t* fjobs;             // [B] the jobs that go through the level sweep
  Frame* frames;               // [B][MAXF]
  uint16_t* fbind;             // [B][MAXF][max_ph] what each frame's placeholders stand for (sets of the chart)
  uint32_t* frame_ctr;         // [B] frames of the job so far
  uint32_t* st32;              // [B][st_stride] the fill's level sweep: the set each trie node leads to (see fill_kernel)
  ulonglong2* req2;            // [req2_cap] its queue of transitions to compute, two halves for odd and even depths
  uint32_t req2_cap;
};

struct StateDev {
  uint32_t B;
  uint32_t ctx_mode;          // 1: this is the view of a root sweep (see RootDev)
  uint32_t gen;               // generation of the sweep's per-job hashes and queue tags (1 .. 65535)
  uint32_t gen_ctx;           // generation of the context-dependent walk's tables
  uint32_t poll_limit_shift;  // bounded waits give up after 2^shift polls
  uint32_t time_steps;        // count the SM cycles spent inside Earley steps (costs a few per cent of the sweep)
  uint32_t chart_words;       // capacity of one private chart buffer
  uint32_t cache_on;
  uint32_t* full_flag;        // host-mapped word (or nullptr): set when the state cache or its mask rows have no room left
  uint32_t max_states, ht_mask, max_mask_rows;
  uint64_t pool_base, pool_words;   // word offsets into arena / size of the pool (the generation in use)
  uint64_t pool_lo;                 // where chart storage of the cache begins (both generations lie above it)
  uint32_t mrow_base;               // first cached mask row of the generation in use (an index into mask_rows)
  uint8_t* st_ref;                  // [max_states] the entry was found again after it was made (it survives the next emptying)
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
  RootDev rt;
  CtxDev cx;
};

constexpr int32_t TR_REJECT = -2;                 // tr_val: the token cannot follow
constexpr int32_t TR_UNSET = (int32_t)0x80808080;  // tr_val: not written yet (the arrays are filled with byte 0x80)
constexpr int32_t MASK_ZERO = -1;       // row_mask: all-zero mask (broken row)
constexpr int32_t MASK_EOS_ONLY = -2;   // row_mask: finished row
constexpr int32_t MASK_ALIAS0 = -10;    // row_mask <= MASK_ALIAS0: same mask as row (MASK_ALIAS0 - x)

}  // namespace fmt
