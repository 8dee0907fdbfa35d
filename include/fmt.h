/*
 * fmt - vocabulary masking for grammar-constrained decoding on one NVIDIA B200 (sm_100a).
 *
 * The library implements the per-step token mask of "Earley-Driven Dynamic Pruning for
 * Efficient Structured Decoding" (ZapFormat / Formatron): every vocabulary token's bytes are
 * fed through each sequence's pruned Earley chart and the token is valid iff the chart stays
 * non-empty (Sections 3.2, 3.3, 4.1, 4.2 of the paper).
 *
 * Conventions
 *  - Every function returns fmt_status (FMT_OK = 0).  No exception crosses this boundary.
 *    fmt_last_error() gives a thread-local message for the last non-OK return.
 *  - Pointers named *_dev are DEVICE pointers, all others are HOST pointers.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All device
 *    work is enqueued on it; unless stated otherwise a call does not synchronize.
 *  - Handles (fmt_grammar, fmt_state) are owned by the library and freed by the matching
 *    destroy.  Caller buffers are never freed or kept beyond the stream work of the call.
 *  - Per-row problems (a rejected token, a finished row, a capacity overflow) are data: they
 *    are written to the caller's status array and the call itself still returns FMT_OK.
 *  - One fmt_state must be used from one stream at a time.
 *
 * Grammar text (Section 3.1: rules A -> alpha over terminals and non-terminals; terminals here
 * are single bytes or byte classes, i.e. the grammar is scannerless):
 *     name ::= alternative ( "|" alternative )*
 *     items: "literal"  [class]  [^negated]  name  ( group )  postfix * + ?   # comment
 *     escapes: \xHH \n \r \t \\ \" \] \- \^ ; "" is the empty string
 *
 * Mask format (Section 3.3): ceil(V/32) uint32 words per row; bit (t & 31) of word (t >> 5)
 * is 1 iff token t may come next; padding bits are 0.  The EOS token is valid iff the bytes so
 * far form a complete sentence.  Any other token with no bytes is never valid.
 */
#ifndef FMT_H_
#define FMT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FMT_OK = 0,
  FMT_ERR_INVALID_ARG = 1,
  FMT_ERR_GRAMMAR_SYNTAX = 2,
  FMT_ERR_UNDEFINED_SYMBOL = 3,
  FMT_ERR_EMPTY_LANGUAGE = 4,
  FMT_ERR_OOM = 5,
  FMT_ERR_CUDA = 6,
  FMT_ERR_CAPACITY = 7,       /* a chart, set or table outgrew its configured capacity */
  FMT_ERR_TOKEN_REJECTED = 8, /* per row: the token is not valid in the current state */
  FMT_ERR_FINISHED = 9        /* per row: EOS was already taken */
} fmt_status;

typedef enum { FMT_BF16 = 0, FMT_FP32 = 1 } fmt_dtype;

typedef struct fmt_grammar fmt_grammar;
typedef struct fmt_state fmt_state;

/* Options of fmt_compile.  Zero-initialise, then set what you need; 0 means "default". */
typedef struct {
  uint32_t host_only;        /* 1: build the tables on the host only (no device needed; the
                                grammar can be inspected but no state can be created) */
  uint32_t no_dfa_terminals; /* 1: keep every non-terminal as rules.  By default a non-terminal whose language is
                                regular (everything it reaches recurses only at the right end, or only at the left
                                end, of its rules - what `*` and `+` turn into) and that is used from a rule that
                                is not, is compiled into one deterministic automaton over the bytes (Section 4.1:
                                terminals as regular languages run as state machines): inside it an Earley item is
                                "automaton state q, begun in set o", a byte is one table look-up, and Predict and
                                Complete run only where the automaton begins and where it accepts.  The language
                                and the masks are the same either way; pruned charts differ in their items */
  uint32_t reserved[6];
} fmt_compile_options;

/* Options of fmt_state_create.  Zero-initialise; 0 means "default". */
typedef struct {
  uint32_t cache_disable;     /* 1: no state cache: every fill recomputes its mask */
  uint32_t max_states;        /* state-cache entries (default 262144) */
  uint32_t max_mask_rows;     /* cached mask rows (default 32768; each holds ceil(V/32) words) */
  uint32_t chart_words;       /* capacity of one row's chart in uint32 words (default 65536) */
  uint64_t pool_words;        /* uint32 words of chart storage for the cache (default 192 Mi) */
  uint32_t sweep_states;       /* distinct Earley sets one mask computation may create while it
                                 sweeps the vocabulary (default: 4 Mi / batch, within 2048..32768) */
  uint32_t roots_enable;       /* 1: keep the context-independent mask cache (Section 4.3): last Earley sets
                                 with their origins made anonymous, each swept once over the vocabulary, so
                                 that rows in the same situation share table look-ups and run Earley steps
                                 only where the answer depends on their own chart.  Off by default: it cuts
                                 the Earley steps per computed row several times but costs about 1 GB of
                                 device memory and, on the workloads measured, more time per fill than it
                                 saves (each trie depth still waits for its slowest step) */
  uint32_t max_roots;          /* entries of the context-independent mask cache (default 4096; each
                                 holds one mask row of ceil(V/32) words) */
  uint32_t root_max_items;     /* a last Earley set with more items than this gets no entry (default and maximum 1024) */
  uint32_t root_max_origins;   /* nor one whose items start in more distinct earlier sets (default 16) */
  uint32_t wait_limit_log2;    /* every wait inside a kernel is a poll that gives up after 2^this many
                                 polls (0 = defaults, 2^21..2^24); see fmt_state_set_wait_limit */
  uint32_t cache_keep_when_full; /* 0: when the state cache has no room for a new entry (states, chart
                                 storage or mask rows), the next fmt_state_advance turns it over: the cache's
                                 storage exists twice, the other copy becomes the one in use, the rows' current
                                 charts are entered again, and so is - with its mask row - every entry that was
                                 found again at least once after it was made (a second chance for what is in
                                 use; what was met once goes).  max_states, max_mask_rows and pool_words are the
                                 capacities of ONE copy.  1: one copy only; when it is full the cache keeps
                                 what it has and takes no new entries */
} fmt_state_options;

typedef struct {
  uint32_t n_nonterminals;   /* after useless-rule removal, including the augmented start */
  uint32_t n_rules;          /* productions kept (empty ones are folded into nullability) */
  uint32_t n_dotted;         /* dotted-rule positions D */
  uint32_t n_classes;        /* distinct byte classes */
  uint32_t n_nullable;       /* nullable non-terminals */
  uint32_t vocab_size;       /* V */
  uint32_t mask_words;       /* ceil(V/32) */
  uint32_t trie_nodes;       /* T, including the root */
  uint32_t trie_depth;       /* longest token in bytes */
  uint32_t n_byte_classes;   /* bytes fall into this many classes that no grammar terminal tells apart */
  uint32_t n_empty_tokens;   /* tokens with no bytes (EOS included) */
  uint32_t start_nullable;   /* 1 if the empty string is a sentence */
  uint32_t n_automata;       /* regular non-terminals that run as deterministic automata (Section 4.1) */
  uint32_t n_automaton_states; /* their states, all together (each is one dotted-rule id, counted in n_dotted) */
} fmt_grammar_info;

typedef struct {
  uint64_t steps_advanced;     /* row-advances that changed a chart */
  uint64_t fills;              /* rows asked for a mask */
  uint64_t fills_computed;     /* rows whose mask was computed by the trie sweep */
  uint64_t fills_from_cache;   /* rows served from a cached mask */
  uint64_t fills_shared;       /* rows that shared another row's mask computed in the same call */
  uint64_t states_cached;      /* distinct pruned charts held by the cache */
  uint64_t mask_rows_cached;
  uint64_t pool_words_used;
  uint64_t chart_items_max;    /* largest pruned chart seen (items) */
  uint64_t chart_sets_max;     /* most live Earley sets seen in one chart */
  uint64_t capacity_errors;
  uint64_t big_mode_units;     /* times a warp of the trie sweep switched to its large scratch area */
  uint64_t sweep_transitions;   /* Earley steps (scan + complete + predict) done by the trie sweep */
  uint64_t sweep_states;        /* distinct Earley sets created by the trie sweep */
  uint64_t advances_cached;     /* row-advances answered by the transition cache (no Earley step run) */
  uint64_t roots;               /* entries of the context-independent mask cache */
  uint64_t root_sweeps;         /* vocabulary sweeps done to fill such entries (one per entry) */
  uint64_t rows_mask_only;      /* computed rows answered by their entry's mask alone (nothing in their state mattered) */
  uint64_t rows_from_root;      /* computed rows swept over the vocabulary starting from such an entry */
  uint64_t rows_plain;          /* computed rows swept from their own chart's last set (no usable entry) */
  uint64_t walk_transitions;    /* Earley steps run for context-dependent transitions of those sweeps */
  uint64_t walk_states;         /* distinct Earley sets they created */
  uint64_t walk_frames;         /* of those, sets that were themselves known entries (what follows them is
                                   looked up in the entry's transition table again instead of computed) */
  uint64_t fills_aborted;       /* fills given up because a bounded wait ran out (their rows got all-zero masks) */
  uint64_t device_bytes;        /* device memory fmt_state_create allocated for this state */
  uint64_t earley_step_cycles;  /* SM cycles spent inside the Earley steps of fills, summed over warps
                                   (divide by sweep_transitions + walk_transitions for a step's latency) */
  uint64_t advance_chart_words; /* uint32 words of charts read and written by fmt_state_advance */
  uint64_t diag[16];            /* where capacity errors and expired waits came from: [0] a row's table of
                                   Earley sets full, [1] the fill's item pool full, [2] a set beyond the large
                                   per-warp scratch, [3] a work queue full, [4] wait for a transition another
                                   warp computes, [5] wait for queued work, [6] wait for the other thread
                                   blocks, [7] a context-independent entry that could not be kept;
                                   [8..15] the same for the sweeps that fill such entries */
  uint64_t cache_flushes;       /* times the state cache was turned over because it had no room left */
} fmt_stats;

/*
 * Build the device tables of a grammar and the byte trie of a vocabulary.
 * Paper: Section 3.1 (CFG), Section 4.5 (useless rules removed, null rules folded into the
 * prediction tables), Section 4.1 (the vocabulary is what is checked every step).
 *   ebnf, ebnf_len    grammar text (host), need not be NUL-terminated
 *   start_rule        NUL-terminated name of the start rule
 *   vocab_bytes       concatenated token bytes (host); vocab_offsets has V+1 entries, token t
 *                     is vocab_bytes[vocab_offsets[t] .. vocab_offsets[t+1])
 *   eos_token_id      id of the end-of-sequence token, or -1 for none
 *   opt               may be NULL
 * Errors: INVALID_ARG, GRAMMAR_SYNTAX, UNDEFINED_SYMBOL, EMPTY_LANGUAGE (the start rule derives
 * no string), CAPACITY (more than 65535 dotted rules, more than 4096 non-terminals, or a token
 * longer than 32 bytes), OOM, CUDA.
 * The grammar is immutable and may be shared by any number of states.
 */
fmt_status fmt_compile(const char* ebnf, size_t ebnf_len, const char* start_rule, const uint8_t* vocab_bytes,
                       const uint64_t* vocab_offsets, uint32_t V, int32_t eos_token_id,
                       const fmt_compile_options* opt, fmt_grammar** out);
void fmt_grammar_destroy(fmt_grammar* g);

/*
 * A JSON schema as the grammar (the paper's JSON-Schema task, Section 5.1, takes schemas; it leaves
 * the translation to its front end and fixes none, so the rules below are this library's).
 * fmt_json_schema_to_ebnf writes grammar text in the dialect fmt_compile reads, start rule "root":
 * min(cap_bytes, size) bytes to `out` (may be NULL; no terminating NUL) and the full size to
 * *size_bytes.  fmt_compile_json_schema is that followed by fmt_compile.
 * A schema node may hold: "type" (object, array, string, number, integer, boolean, null, or a list
 * of them), "properties" with "required" (members come in the order written; a member that is not
 * required may be left out; no other member is allowed), "items" and "minItems" (0 or 1), "enum",
 * "const", "anyOf" / "oneOf" (both read as "any of"), "$ref" to "#/$defs/NAME" or
 * "#/definitions/NAME" (may be recursive).  A node with none of these accepts any JSON value.
 * Annotations (title, description, default, examples, $schema, $id) are skipped; any other
 * keyword is refused with FMT_ERR_GRAMMAR_SYNTAX rather than silently ignored.  White space is
 * allowed wherever JSON allows it; strings are RFC 8259 strings in well-formed UTF-8.
 */
fmt_status fmt_json_schema_to_ebnf(const char* schema, size_t schema_len, char* out, size_t cap_bytes, size_t* size_bytes);
fmt_status fmt_compile_json_schema(const char* schema, size_t schema_len, const uint8_t* vocab_bytes,
                                   const uint64_t* vocab_offsets, uint32_t V, int32_t eos_token_id,
                                   const fmt_compile_options* opt, fmt_grammar** out);

/* Sizes of the compiled grammar (host data; works for host_only grammars too). */
fmt_status fmt_grammar_get_info(const fmt_grammar* g, fmt_grammar_info* out);

/*
 * Run automaton k (0 .. fmt_grammar_info.n_automata - 1; see fmt_compile_options.no_dfa_terminals) over
 * `bytes` on the host, for inspection and tests: *accepted = 1 iff the bytes are a sentence of the regular
 * non-terminal the automaton stands for, whose name (as in the grammar text; helper non-terminals made
 * by `*`, `+`, `?` and groups carry a `~`) is copied to name_out, NUL-terminated, if name_out is not NULL.
 */
fmt_status fmt_grammar_automaton_match(const fmt_grammar* g, uint32_t k, const uint8_t* bytes, size_t len, int* accepted,
                                       char* name_out, size_t name_cap);

/*
 * Copy one host-side table of the compiled grammar, for inspection and tests.
 *   which: 0 trie child_off [T+1] u32   1 trie node_byte [T] u8    2 trie parent [T] u32
 *          3 trie tok_off [T+1] u32     4 trie tok_ids u32         5 level offsets [depth+2] u32
 *          6 nullable flags [N] u8      7 item info [D] u32        8 item lhs [D] u16
 *          9 tok_node [V] u32 (node where a token ends, 0xFFFFFFFF if it has no bytes)
 *         10 byte class of each byte [256] u8
 *         11 automata: transitions [states][byte classes] u16 (target state | 0x4000 target has transitions |
 *            0x8000 target accepts, 0xFFFF none)   12 accepting flag per state u8   13 start state per automaton u32
 * Writes min(cap_bytes, size) bytes to `out` (may be NULL) and the full size to *size_bytes.
 */
fmt_status fmt_grammar_copy_table(const fmt_grammar* g, int which, void* out, size_t cap_bytes, size_t* size_bytes);

/*
 * Create `batch` sequences, all at the start of the grammar (Earley set S[0], Section 3.2).
 * Runs a small kernel on `stream` and synchronizes it once.  opt may be NULL.
 * Device memory: everything the state will ever use is allocated here (fmt_stats.device_bytes reports it;
 * no later call allocates).  With the default options it is about 3.7 GB for batch 8 and 5.3-6.5 GB for
 * batch 64-256 with a 128 K-152 K vocabulary: 2 x 0.8 GB of chart storage for the state cache (pool_words,
 * two generations: see cache_keep_when_full), 2 x max_mask_rows x ceil(V/32) words of cached masks
 * (2 x 0.5-0.6 GB), batch x 3 private chart buffers of
 * chart_words words, and the fills' working tables (per row a table of up to sweep_states Earley sets,
 * one 16-bit entry per row and trie node, a 0.5 GB pool for the sets' items); the context-independent
 * cache (roots_enable) adds about 1 GB.  A cached state costs its chart (0.8-3.4 KB in the measured
 * workloads) plus, once a mask has been computed for it, one mask row of ceil(V/32) words.
 */
fmt_status fmt_state_create(const fmt_grammar* g, uint32_t batch, const fmt_state_options* opt, void* stream,
                            fmt_state** out);
void fmt_state_destroy(fmt_state* s);

/* Put rows `rows_dev[0..n)` (DEVICE array of row indices; NULL = rows 0..n-1) back to the start. */
fmt_status fmt_state_reset(fmt_state* s, const uint32_t* rows_dev, uint32_t n, void* stream);

/*
 * Advance every row by its chosen token (Section 3.2 scan / complete / predict per byte, with
 * the Compact step of Section 4.2.3 between complete and predict; the resulting pruned chart
 * is looked up in the state cache, Section 5.2 "state cache").  With the cache on, the outcome of
 * advancing a cached chart by a token - the next chart's cache id, or "rejected" - is remembered
 * too, so the same (chart, token) pair later costs one table look-up instead of Earley steps.
 *   token_ids_dev  [batch] int32 on the device; -1 leaves the row alone
 *   status_dev     [batch] int32 on the device or NULL; receives FMT_OK, FMT_ERR_TOKEN_REJECTED
 *                  (row unchanged), FMT_ERR_FINISHED, FMT_ERR_INVALID_ARG (id out of range) or
 *                  FMT_ERR_CAPACITY (row unchanged; its later masks are all-zero)
 * Taking EOS in an accepting state finishes the row: its mask is then the EOS bit alone.
 */
fmt_status fmt_state_advance(fmt_state* s, const int32_t* token_ids_dev, int32_t* status_dev, void* stream);

/*
 * Jump-ahead: per row, the run of bytes that every continuation of the row's text must begin with.
 * (Section 5.1 evaluates a JSON-Schema task, where keys, quotes and punctuation between the values are
 * fixed by the schema; the paper names no such call.  A server may append the run's tokens without
 * sampling.)  As long as the text so far is not a sentence of the grammar (EOS is not valid) and exactly
 * one byte can follow it, that byte joins the run and the row's chart is stepped over it, in scratch
 * memory: the row itself does not change.
 *   bytes_dev     device output, row r's run at bytes_dev[r * stride_bytes ..]; bytes beyond the run's
 *                 length are left as they were
 *   stride_bytes  >= max_len
 *   len_dev       device output, [batch] uint32: the run's length, 0 .. max_len; 0 for finished or
 *                 broken rows.  A run that reaches max_len, or whose Earley sets outgrow the scratch,
 *                 is cut there: every prefix of a forced run is forced, so a shorter answer is still right
 *   max_len       at most FMT_MAX_FORCED_BYTES (larger values are clamped); call again after advancing
 *                 the row for longer runs
 */
#define FMT_MAX_FORCED_BYTES 32
fmt_status fmt_state_forced_bytes(fmt_state* s, uint8_t* bytes_dev, size_t stride_bytes, uint32_t* len_dev, uint32_t max_len,
                                  void* stream);

/*
 * Write the mask of every row (Sections 3.3, 4.1): mask_dev[row * stride_words + w].
 * stride_words >= ceil(V/32).  Rows whose pruned chart is in the state cache copy the cached
 * mask; the others sweep the vocabulary trie.
 */
fmt_status fmt_fill_mask(fmt_state* s, uint32_t* mask_dev, size_t stride_words, void* stream);

/*
 * Section 3.3: set the logits of invalid tokens to -inf (bf16 0xFF80, fp32 0xFF800000); valid
 * entries keep their bits.  logits_dev[row * row_stride_elems + t], t < V.
 */
fmt_status fmt_apply_mask(const uint32_t* mask_dev, size_t stride_words, void* logits_dev, fmt_dtype dtype,
                          uint32_t batch, uint32_t V, size_t row_stride_elems, void* stream);

/* fmt_fill_mask followed by fmt_apply_mask without a second pass over the mask in HBM:
 * the logits are masked straight from the cached mask rows.  mask_dev may be NULL. */
fmt_status fmt_fill_and_apply(fmt_state* s, uint32_t* mask_dev_or_null, size_t stride_words, void* logits_dev,
                              fmt_dtype dtype, size_t row_stride_elems, void* stream);

/* Forget every cached chart and mask of the state cache (rows keep their current charts).  The
 * context-independent mask cache (Section 4.3) is knowledge about the grammar and the vocabulary,
 * not about the sequences, and stays; fmt_state_ci_cache_clear forgets that one. */
fmt_status fmt_state_cache_clear(fmt_state* s, void* stream);
fmt_status fmt_state_ci_cache_clear(fmt_state* s, void* stream);

/* Every wait inside a kernel of this library (for another thread block, for a queued work item, for
 * a transition another warp is computing) is a poll with an iteration limit; a wait that runs out
 * makes the fill give up: its computed rows get all-zero masks, fmt_stats.fills_aborted counts it,
 * nothing hangs and the next fill starts afresh.  log2_polls = 0 restores the defaults.  (A test
 * aid: with a tiny limit the give-up path can be taken without anything being wrong.) */
fmt_status fmt_state_set_wait_limit(fmt_state* s, uint32_t log2_polls);

/* Per-row summary, written to host arrays (any may be NULL); synchronizes `stream`.
 *   accepting[batch] u8, finished[batch] u8 (1 finished, 2 broken by a capacity error),
 *   n_sets[batch] u32, n_items[batch] u32, state_id[batch] i32 (-1 = not in the cache) */
fmt_status fmt_state_query(fmt_state* s, uint8_t* accepting, uint8_t* finished, uint32_t* n_sets,
                           uint32_t* n_items, int32_t* state_id, void* stream);

/* Copy the pruned chart of one row to the host, for inspection and tests; synchronizes `stream`.
 * Layout (uint32 words): [0] live sets m, [1] items, [2] flags (bit 0 accepting), [3],[4] hash,
 * [5] total words, [6],[7] unused, then set_off[m+1], then the items (origin << 16 | dotted rule).
 * Writes min(cap_words, total) words to `out` (may be NULL) and the total to *n_words. */
fmt_status fmt_state_copy_chart(fmt_state* s, uint32_t row, uint32_t* out, size_t cap_words, size_t* n_words,
                                void* stream);

/* Raw device counters of the state (which = 0) or of its sweeps of context-independent entries
 * (which = 1), for inspection and tests: min(cap_words, total) uint32 words to `out`, the total to
 * *n_words; synchronizes `stream`.  The layout is the library's own (csrc/device_tables.h). */
fmt_status fmt_state_copy_counters(fmt_state* s, int which, uint32_t* out, size_t cap_words, size_t* n_words, void* stream);

/* Counters since creation; synchronizes `stream`. */
fmt_status fmt_get_stats(fmt_state* s, fmt_stats* out, void* stream);

/* Kernel timing with CUDA events on the caller's stream (no counterpart in the paper: a
 * measurement aid).  While enabled, every fmt_state_advance, both halves of every fill (first the work
 * on context-independent entries: finding each row's entry and sweeping the new ones; then the trie
 * sweep of the rows) and every logits-masking kernel of this state are bracketed by pairs of events (up
 * to 16384 pairs per kind, later launches are not timed).  fmt_state_read_profile synchronizes those
 * events, adds up the elapsed times and forgets them.  `enable` is a set of bits: 1 = those events;
 * 2 = count the SM cycles that warps spend inside Earley steps (fmt_stats.earley_step_cycles; reading
 * the cycle counter around every step slows the sweeps by several per cent, so it is a switch). */
typedef struct {
  double advance_ms, sweep_ms, apply_ms;
  uint64_t advance_launches, sweep_launches, apply_launches;
  double roots_ms;         /* the fills' work on context-independent entries */
  uint64_t roots_launches;
} fmt_profile;
fmt_status fmt_state_set_profiling(fmt_state* s, int enable);
fmt_status fmt_state_read_profile(fmt_state* s, fmt_profile* out);
/* The same measurements launch by launch, before fmt_state_read_profile forgets them: kind 0 advance,
 * 1 trie sweep, 2 logits masking, 3 the fills' work on context-independent entries.  Writes up to `cap`
 * durations in milliseconds to ms_out (may be NULL) and the number recorded to *n. */
fmt_status fmt_state_read_profile_series(fmt_state* s, int kind, float* ms_out, size_t cap, size_t* n);

/*
 * Masks for up to FMT_NOALLOC_MAX_CHARTS pruned charts without any memory allocation.
 * (The paper has no counterpart; this is a convenience of this library.)
 *
 * Who needs it: code that must not call cudaMalloc / cudaFree while it runs - a serving loop
 * whose device memory is entirely owned by a caching allocator or handed out up front, a
 * real-time or library context where an allocation may synchronize the device or fail under
 * memory pressure, a plugin that may only launch kernels.  fmt_fill_mask itself never allocates,
 * but it needs an fmt_state, whose creation allocates gigabytes (fmt_stats.device_bytes).  This call needs no
 * fmt_state: it sweeps the vocabulary trie for charts the caller already holds in device memory
 * (in the layout fmt_state_copy_chart documents) and uses a fixed scratch array that is part of
 * the loaded library image (about 55 MB of device memory on every GPU that loads the library,
 * held until the process exits).
 *
 *   g              a grammar compiled for the current device
 *   charts_dev     device memory holding the charts
 *   chart_offsets  HOST array of n+1 word offsets into charts_dev: chart r occupies words
 *                  [chart_offsets[r], chart_offsets[r+1])
 *   n              number of charts, at most FMT_NOALLOC_MAX_CHARTS, and n x (trie nodes of the
 *                  vocabulary) at most 8 Mi (beyond either limit: FMT_ERR_CAPACITY)
 *   mask_dev       device output, n rows of exactly ceil(V/32) words (dense, no extra stride)
 *   status_dev     device output or NULL, n int32: FMT_OK, FMT_ERR_INVALID_ARG (the chart does not fit
 *                  its slot, its sets' offsets decrease, or an item names a dotted rule or a set that
 *                  does not exist; such a chart is not swept and its mask is all-zero) or
 *                  FMT_ERR_CAPACITY (the Earley sets met while sweeping the vocabulary outgrew the
 *                  fixed scratch, or a bounded wait inside the sweep ran out, which gives up every
 *                  chart of the call; that row's mask is all-zero)
 *
 * The first call on each device looks up the scratch array's device address and raises the
 * kernels' shared-memory limit; make that first call outside any stream capture.  Every call on
 * a device uses the same scratch array: calls that may overlap on the GPU (different streams,
 * different host threads) race and must be serialized by the caller.  The call enqueues work on
 * `stream` and does not synchronize; it calls no cudaMalloc, cudaFree or other allocating routine.
 */
#define FMT_NOALLOC_MAX_CHARTS 64
fmt_status fmt_fill_mask_noalloc(const fmt_grammar* g, const uint32_t* charts_dev, const uint64_t* chart_offsets,
                                 uint32_t n, uint32_t* mask_dev, int32_t* status_dev, void* stream);

const char* fmt_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FMT_H_ */
