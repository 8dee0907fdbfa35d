// Host-side result of compiling a grammar and a vocabulary: flat integer tables that are
// uploaded to the device as they are.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace fmt {

// item info word: bits 31..30 kind, bit 29 "post-dot non-terminal is nullable", bits 23..16 how many
// nullable non-terminals follow the dot in a row (the dot may move over them), bits 15..0 argument
//   END : argument = left-hand side        (dot at the end of the rule)
//   TERM: argument = byte-class id         (post-dot symbol is a terminal)
//   NT  : argument = non-terminal id       (post-dot symbol is a non-terminal)
//   DFA : argument = automaton state      (the item is inside a regular non-terminal run as an automaton)
enum : uint32_t { KIND_END = 0u, KIND_TERM = 1u, KIND_NT = 2u, KIND_DFA = 3u };
constexpr uint32_t INFO_KIND_SHIFT = 30;
constexpr uint32_t INFO_NULLABLE = 1u << 29;
constexpr uint32_t INFO_ARG_MASK = 0xFFFFu;
constexpr uint32_t INFO_SKIP_SHIFT = 16, INFO_SKIP_MASK = 0xFFu;
constexpr uint32_t ITEM_START = 0;   // $ -> . start
constexpr uint32_t ITEM_ACCEPT = 1;  // $ -> start .
constexpr uint32_t MAX_TOKEN_BYTES = 32;
constexpr uint32_t MAX_NONTERMINALS = 4096;

struct CompileError {
  int code;
  std::string msg;
};

struct HostTables {
  // ---- grammar (Section 3.1; reduced as in Section 4.5)
  uint32_t N = 0, P = 0, D = 0, C = 0, Nw = 0, n_nullable = 0;
  bool start_nullable = false;
  std::vector<uint32_t> info;          // [D]
  std::vector<uint16_t> lhs;           // [D] left-hand side of the item's rule
  std::vector<uint8_t> skip;           // [D] how many nullable non-terminals follow the dot in a row
  std::vector<uint32_t> class_bits;    // [C][8] 256-bit byte classes
  std::vector<uint32_t> nt_closure;    // [N][Nw] non-terminals predicted (transitively) with Y
  std::vector<uint32_t> direct_off;    // [N+1]
  std::vector<uint16_t> direct_items;  // start items of each non-terminal's rules, dots moved over
                                       // leading nullable symbols, completed items left out
  std::vector<uint8_t> eq_of_byte;     // [256] bytes that belong to the same byte classes share a number
  uint32_t n_eq = 0;                   // how many such equivalence classes of bytes there are
  // regular non-terminals run as deterministic automata (Section 4.1's regular terminals): item id
  // dfa_first + g is state g; dfa_trans[g][byte class] = target state | 0x4000 (the target has transitions
  // of its own) | 0x8000 (the target accepts), or 0xFFFF
  uint32_t dfa_first = 0, dfa_states = 0;
  std::vector<uint16_t> dfa_trans;     // [dfa_states][n_eq]
  std::vector<uint16_t> dfa_done;      // [dfa_states] id of the completed item of the state's non-terminal
  std::vector<uint32_t> dfa_scan;      // [dfa_states][8] bytes with a transition
  std::vector<uint8_t> dfa_accept;     // [dfa_states]
  std::vector<uint32_t> dfa_nt;        // per automaton: its non-terminal
  std::vector<uint32_t> dfa_start;     // per automaton: its start state
  std::vector<uint8_t> nullable;       // [N]
  std::vector<std::string> nt_names;   // [N]
  // ---- vocabulary trie in CSR form, nodes in breadth-first order (root = 0)
  uint32_t V = 0, Wm = 0, T = 0, depth = 0, n_empty = 0;
  int32_t eos = -1;
  std::vector<uint32_t> child_off;  // [T+1] children of node n are nodes child_off[n]..child_off[n+1]-1
  std::vector<uint8_t> node_byte;   // [T]
  std::vector<uint32_t> parent;     // [T]
  std::vector<uint8_t> node_depth;  // [T]
  std::vector<uint32_t> tok_off;    // [T+1] tokens whose bytes end at node n
  std::vector<uint32_t> tok_ids;
  std::vector<uint32_t> lvl_off;    // [depth+2] nodes of depth L are lvl_off[L]..lvl_off[L+1]-1
  std::vector<uint32_t> tok_node;   // [V] node where the token's bytes end, 0xFFFFFFFF for empty tokens
  std::vector<uint32_t> vocab_off;  // [V+1] byte offsets (32-bit) into vocab_bytes
  std::vector<uint8_t> vocab_bytes;
};

// Grammar text (start rule "root") for the instances of a JSON schema; throws CompileError.
std::string json_schema_to_ebnf(const char* schema, size_t len);

// Both throw CompileError.
void compile_grammar(const char* text, size_t len, const std::string& start, HostTables& out, bool dfa_terminals = true);
void build_trie(const uint8_t* bytes, const uint64_t* offs, uint32_t V, int32_t eos, HostTables& out);

}  // namespace fmt
