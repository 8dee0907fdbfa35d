// Grammar text -> reduced grammar -> flat tables; vocabulary -> CSR byte trie in level order.
//
// Follows the paper's Section 3.1 (rules A -> alpha), Section 4.5 (remove useless rules; handle
// rules deriving the empty string once, at compile time) and Section 4.1 (the whole vocabulary
// is checked each step, hence the trie).  Repetition is desugared into LEFT recursion so that
// the pruned chart of a list does not grow with the list's length (rules of the form A -> B a
// are the ones whose history can be dropped, Section 4.1).
#include <algorithm>
#include <array>
#include <cctype>
#include <cstring>
#include <map>

#include "../../include/fmt.h"
#include "host_tables.h"

namespace fmt {
namespace {

using Bits256 = std::array<uint32_t, 8>;

// ------------------------------------------------------------------------------------ lexer

enum class Tok { Ident, Define, Bar, LParen, RParen, Star, Plus, Question, Literal, Class, End };

struct Lexeme {
  Tok kind;
  std::string text;  // Ident name / Literal bytes
  Bits256 cls;       // Class
  size_t pos;
};

class Lexer {
 public:
  Lexer(const char* s, size_t n) : s_(s), n_(n) {}

  std::vector<Lexeme> run() {
    std::vector<Lexeme> out;
    for (;;) {
      blank();
      if (p_ >= n_) break;
      size_t at = p_;
      unsigned char c = (unsigned char)s_[p_];
      if (c == ':' && p_ + 2 < n_ && s_[p_ + 1] == ':' && s_[p_ + 2] == '=') {
        p_ += 3;
        out.push_back(simple(Tok::Define, at));
      } else if (c == '|') {
        ++p_, out.push_back(simple(Tok::Bar, at));
      } else if (c == '(') {
        ++p_, out.push_back(simple(Tok::LParen, at));
      } else if (c == ')') {
        ++p_, out.push_back(simple(Tok::RParen, at));
      } else if (c == '*') {
        ++p_, out.push_back(simple(Tok::Star, at));
      } else if (c == '+') {
        ++p_, out.push_back(simple(Tok::Plus, at));
      } else if (c == '?') {
        ++p_, out.push_back(simple(Tok::Question, at));
      } else if (c == '"') {
        out.push_back(literal());
      } else if (c == '[') {
        out.push_back(byte_class());
      } else if (isalpha(c) || c == '_') {
        size_t q = p_ + 1;
        while (q < n_ && (isalnum((unsigned char)s_[q]) || s_[q] == '_' || s_[q] == '-')) ++q;
        Lexeme l = simple(Tok::Ident, at);
        l.text.assign(s_ + p_, q - p_);
        out.push_back(l);
        p_ = q;
      } else {
        throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "unexpected byte at offset " + std::to_string(at)};
      }
    }
    out.push_back(simple(Tok::End, n_));
    return out;
  }

 private:
  const char* s_;
  size_t n_, p_ = 0;

  static Lexeme simple(Tok k, size_t at) {
    Lexeme l;
    l.kind = k;
    l.cls.fill(0);
    l.pos = at;
    return l;
  }
  void blank() {
    while (p_ < n_) {
      if (s_[p_] == '#') {
        while (p_ < n_ && s_[p_] != '\n') ++p_;
      } else if (s_[p_] == ' ' || s_[p_] == '\t' || s_[p_] == '\n' || s_[p_] == '\r') {
        ++p_;
      } else {
        return;
      }
    }
  }
  static int hex(unsigned char c) {
    if (c >= '0' && c <= '9') return c - '0';
    c |= 0x20;
    if (c >= 'a' && c <= 'f') return c - 'a' + 10;
    return -1;
  }
  unsigned char escaped() {  // p_ is just past the backslash
    if (p_ >= n_) throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "backslash at end of text"};
    unsigned char c = (unsigned char)s_[p_++];
    if (c == 'n') return 10;
    if (c == 'r') return 13;
    if (c == 't') return 9;
    if (c == 'x') {
      int a = p_ < n_ ? hex((unsigned char)s_[p_]) : -1, b = p_ + 1 < n_ ? hex((unsigned char)s_[p_ + 1]) : -1;
      if (a < 0 || b < 0) throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "bad \\x escape at offset " + std::to_string(p_)};
      p_ += 2;
      return (unsigned char)(a * 16 + b);
    }
    return c;
  }
  Lexeme literal() {
    Lexeme l = simple(Tok::Literal, p_);
    ++p_;
    while (true) {
      if (p_ >= n_) throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "literal not closed (offset " + std::to_string(l.pos) + ")"};
      unsigned char c = (unsigned char)s_[p_++];
      if (c == '"') break;
      l.text.push_back((char)(c == '\\' ? escaped() : c));
    }
    return l;
  }
  Lexeme byte_class() {
    Lexeme l = simple(Tok::Class, p_);
    ++p_;
    bool invert = false;
    if (p_ < n_ && s_[p_] == '^') invert = true, ++p_;
    while (true) {
      if (p_ >= n_) throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "class not closed (offset " + std::to_string(l.pos) + ")"};
      unsigned char c = (unsigned char)s_[p_++];
      if (c == ']') break;
      unsigned lo = (c == '\\') ? escaped() : c, hi = lo;
      if (p_ + 1 < n_ && s_[p_] == '-' && s_[p_ + 1] != ']') {
        ++p_;
        unsigned char e = (unsigned char)s_[p_++];
        hi = (e == '\\') ? escaped() : e;
        if (hi < lo) throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "range out of order (offset " + std::to_string(p_) + ")"};
      }
      for (unsigned b = lo; b <= hi; ++b) l.cls[b >> 5] |= 1u << (b & 31);
    }
    if (invert)
      for (auto& w : l.cls) w = ~w;
    bool any = false;
    for (auto w : l.cls) any |= (w != 0);
    if (!any) throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "empty byte class (offset " + std::to_string(l.pos) + ")"};
    return l;
  }
};

// ------------------------------------------------------------------------------------ parser

// symbol: >= 0 non-terminal id, < 0 terminal class ~id
struct Production {
  int lhs;
  std::vector<int> rhs;
};

class GrammarBuilder {
 public:
  std::vector<std::string> names;
  std::vector<char> defined;
  std::vector<Production> prods;
  std::vector<Bits256> classes;

  int nt(const std::string& name) {
    auto it = ids_.find(name);
    if (it != ids_.end()) return it->second;
    int id = (int)names.size();
    ids_[name] = id;
    names.push_back(name);
    defined.push_back(0);
    return id;
  }
  int lookup(const std::string& name) const {
    auto it = ids_.find(name);
    return it == ids_.end() ? -1 : it->second;
  }
  int fresh(const std::string& hint) {
    std::string nm = hint + "~" + std::to_string(++counter_);
    int id = nt(nm);
    defined[id] = 1;
    return id;
  }
  int terminal(const Bits256& b) {
    auto it = class_ids_.find(b);
    if (it != class_ids_.end()) return ~it->second;
    int id = (int)classes.size();
    classes.push_back(b);
    class_ids_[b] = id;
    return ~id;
  }

 private:
  std::map<std::string, int> ids_;
  std::map<Bits256, int> class_ids_;
  int counter_ = 0;
};

class Parser {
 public:
  Parser(std::vector<Lexeme> lx, GrammarBuilder& b) : lx_(std::move(lx)), b_(b) {}

  void run() {
    if (lx_[0].kind == Tok::End) throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "the grammar has no rules"};
    while (lx_[i_].kind != Tok::End) {
      if (!rule_starts_here())
        throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "expected `name ::=` at offset " + std::to_string(lx_[i_].pos)};
      int lhs = b_.nt(lx_[i_].text);
      b_.defined[lhs] = 1;
      ctx_ = lx_[i_].text;
      i_ += 2;
      alternatives(lhs);
    }
  }

 private:
  std::vector<Lexeme> lx_;
  GrammarBuilder& b_;
  size_t i_ = 0;
  std::string ctx_;

  bool rule_starts_here() const { return lx_[i_].kind == Tok::Ident && lx_[i_ + 1].kind == Tok::Define; }

  void alternatives(int lhs) {
    for (;;) {
      std::vector<int> body = sequence();
      b_.prods.push_back({lhs, body});
      if (lx_[i_].kind == Tok::Bar) {
        ++i_;
        continue;
      }
      break;
    }
  }
  std::vector<int> sequence() {
    std::vector<int> out;
    for (;;) {
      Tok k = lx_[i_].kind;
      if (k == Tok::End || k == Tok::Bar || k == Tok::RParen || rule_starts_here()) break;
      std::vector<int> piece = postfixed();
      out.insert(out.end(), piece.begin(), piece.end());
    }
    return out;
  }
  std::vector<int> postfixed() {
    std::vector<int> unit = primary();
    for (;;) {
      Tok k = lx_[i_].kind;
      if (k == Tok::Star) {  // X -> empty | X unit
        int x = b_.fresh(ctx_);
        std::vector<int> rec{x};
        rec.insert(rec.end(), unit.begin(), unit.end());
        b_.prods.push_back({x, {}});
        b_.prods.push_back({x, rec});
        unit = {x};
      } else if (k == Tok::Plus) {  // X -> unit | X unit
        int x = b_.fresh(ctx_);
        std::vector<int> rec{x};
        rec.insert(rec.end(), unit.begin(), unit.end());
        b_.prods.push_back({x, unit});
        b_.prods.push_back({x, rec});
        unit = {x};
      } else if (k == Tok::Question) {  // X -> empty | unit
        int x = b_.fresh(ctx_);
        b_.prods.push_back({x, {}});
        b_.prods.push_back({x, unit});
        unit = {x};
      } else {
        break;
      }
      ++i_;
    }
    return unit;
  }
  std::vector<int> primary() {
    const Lexeme l = lx_[i_];
    switch (l.kind) {
      case Tok::Literal: {
        ++i_;
        std::vector<int> out;
        for (unsigned char c : l.text) {
          Bits256 one;
          one.fill(0);
          one[c >> 5] = 1u << (c & 31);
          out.push_back(b_.terminal(one));
        }
        return out;
      }
      case Tok::Class:
        ++i_;
        return {b_.terminal(l.cls)};
      case Tok::Ident:
        ++i_;
        return {b_.nt(l.text)};
      case Tok::LParen: {
        ++i_;
        size_t first = b_.prods.size();
        int x = b_.fresh(ctx_);
        alternatives(x);
        if (lx_[i_].kind != Tok::RParen)
          throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "expected ) at offset " + std::to_string(lx_[i_].pos)};
        ++i_;
        // a group with one alternative is spliced in place
        size_t count = 0, where = 0;
        for (size_t p = first; p < b_.prods.size(); ++p)
          if (b_.prods[p].lhs == x) ++count, where = p;
        if (count == 1) {
          std::vector<int> body = b_.prods[where].rhs;
          b_.prods.erase(b_.prods.begin() + (long)where);
          return body;
        }
        return {x};
      }
      default:
        throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "unexpected token at offset " + std::to_string(l.pos)};
    }
  }
};

// ------------------------------------------------------------------------------------ regular non-terminals -> DFAs
//
// Section 4.1 models terminals as regular languages run as finite-state machines inside the chart.
// Here the grammar text has no separate lexical level, so the regular parts are found: a
// non-terminal is regular when, in everything it can reach, recursion is only ever at the right end
// of a rule or only ever at the left end (within each group of mutually recursive non-terminals;
// `*` and `+` are desugared into exactly such rules).  A regular non-terminal that is used from a
// non-regular rule becomes one deterministic automaton over the byte classes; the Earley items inside
// it are "automaton state q, started in set o" and a byte costs one table look-up, with no Predict and
// no Complete until the automaton accepts (then it completes like any non-terminal).

struct Nfa {
  std::vector<std::vector<int>> eps;
  std::vector<std::vector<std::pair<int, int>>> edge;  // (byte class, target)
  int add() {
    eps.emplace_back();
    edge.emplace_back();
    return (int)eps.size() - 1;
  }
};

struct OneDfa {
  int nt = -1;                       // the non-terminal it stands for (builder numbering)
  uint32_t n_states = 0;             // state 0 is the start state
  std::vector<int> trans;            // [n_states][n_eq] target state or -1
  std::vector<char> accepting;       // [n_states]
};

struct RegularInfo {
  std::vector<int> scc_of;           // per non-terminal
  std::vector<std::vector<int>> scc_members;
  std::vector<int> scc_kind;         // 0 not regular, 1 no recursion, 2 right-linear, 3 left-linear
  std::vector<char> regular;         // per non-terminal
};

constexpr size_t NFA_STATE_CAP = 60000, DFA_STATE_CAP = 6000;

class DfaBuilder {
 public:
  DfaBuilder(const std::vector<Production>& rules, size_t n_nt, const std::vector<Bits256>& classes,
             const std::vector<uint8_t>& eq_of_byte, uint32_t n_eq)
      : rules_(rules), n_nt_(n_nt), classes_(classes), n_eq_(n_eq) {
    by_lhs_.resize(n_nt);
    for (size_t i = 0; i < rules.size(); ++i) by_lhs_[rules[i].lhs].push_back((int)i);
    rep_.assign(n_eq, 0);
    for (int b = 255; b >= 0; --b) rep_[eq_of_byte[b]] = (uint8_t)b;
    classify();
  }
  const RegularInfo& info() const { return info_; }

  // The automaton of regular non-terminal x, minimised; false if it outgrows the caps.
  bool build(int x, OneDfa& out) {
    Nfa n;
    too_big_ = false;
    const int s = n.add(), t = n.add();
    instantiate(n, x, s, t);
    if (too_big_) return false;
    return determinise(n, s, t, out) && (out.nt = x, true);
  }

 private:
  const std::vector<Production>& rules_;
  size_t n_nt_;
  const std::vector<Bits256>& classes_;
  uint32_t n_eq_;
  std::vector<std::vector<int>> by_lhs_;
  std::vector<uint8_t> rep_;  // one byte of every equivalence class
  RegularInfo info_;
  bool too_big_ = false;

  // ---- strongly connected components of "A uses B" (Tarjan, iterative enough for grammar sizes: recursion depth = chain length)
  void classify() {
    const int n = (int)n_nt_;
    info_.scc_of.assign(n, -1);
    std::vector<int> index(n, -1), low(n, 0), stack;
    std::vector<char> on(n, 0);
    int counter = 0;
    struct Frame {
      int v;
      size_t rule, sym;
    };
    for (int root = 0; root < n; ++root) {
      if (index[root] >= 0 || by_lhs_[root].empty()) continue;
      std::vector<Frame> call{{root, 0, 0}};
      index[root] = low[root] = counter++;
      stack.push_back(root), on[root] = 1;
      while (!call.empty()) {
        Frame& f = call.back();
        bool descended = false;
        while (f.rule < by_lhs_[f.v].size() && !descended) {
          const Production& p = rules_[by_lhs_[f.v][f.rule]];
          while (f.sym < p.rhs.size()) {
            const int w = p.rhs[f.sym++];
            if (w < 0 || by_lhs_[w].empty()) continue;
            if (index[w] < 0) {
              index[w] = low[w] = counter++;
              stack.push_back(w), on[w] = 1;
              call.push_back({w, 0, 0});
              descended = true;
              break;
            }
            if (on[w]) low[f.v] = std::min(low[f.v], index[w]);
          }
          if (!descended) ++f.rule, f.sym = 0;
        }
        if (descended) continue;
        const int v = f.v;
        call.pop_back();
        if (!call.empty()) low[call.back().v] = std::min(low[call.back().v], low[v]);
        if (low[v] == index[v]) {
          const int id = (int)info_.scc_members.size();
          info_.scc_members.emplace_back();
          for (;;) {
            const int w = stack.back();
            stack.pop_back(), on[w] = 0;
            info_.scc_of[w] = id;
            info_.scc_members[id].push_back(w);
            if (w == v) break;
          }
        }
      }
    }
    // components come out callees first: a component's kind and whether all it uses is regular
    const int m = (int)info_.scc_members.size();
    info_.scc_kind.assign(m, 0);
    info_.regular.assign(n, 0);
    for (int c = 0; c < m; ++c) {
      bool right_ok = true, left_ok = true, recursive = false, uses_ok = true;
      for (int a : info_.scc_members[c])
        for (int r : by_lhs_[a]) {
          const Production& p = rules_[r];
          int inside = 0;
          for (size_t k = 0; k < p.rhs.size(); ++k) {
            const int w = p.rhs[k];
            if (w < 0) continue;
            if (info_.scc_of[w] == c) {
              ++inside;
              if (k + 1 != p.rhs.size()) right_ok = false;
              if (k != 0) left_ok = false;
            } else if (!info_.regular[w]) {
              uses_ok = false;
            }
          }
          if (inside) recursive = true;
          if (inside > 1) right_ok = left_ok = false;
        }
      int kind = 0;
      if (uses_ok) kind = !recursive ? 1 : right_ok ? 2 : left_ok ? 3 : 0;
      info_.scc_kind[c] = kind;
      for (int a : info_.scc_members[c]) info_.regular[a] = kind != 0;
    }
  }

  // ---- Thompson-style construction: non-terminal x between NFA states `from` and `to`
  void chain(Nfa& n, int a, const std::vector<int>& syms, size_t lo, size_t hi, int b) {
    if (too_big_) return;
    if (lo == hi) {
      n.eps[a].push_back(b);
      return;
    }
    int cur = a;
    for (size_t k = lo; k < hi; ++k) {
      const int nxt = (k + 1 == hi) ? b : n.add();
      if (syms[k] < 0) n.edge[cur].push_back({~syms[k], nxt});
      else instantiate(n, syms[k], cur, nxt);
      cur = nxt;
    }
  }
  void instantiate(Nfa& n, int x, int from, int to) {
    if (n.eps.size() > NFA_STATE_CAP) too_big_ = true;
    if (too_big_) return;
    const int c = info_.scc_of[x];
    const int kind = info_.scc_kind[c];
    if (kind == 1) {
      for (int r : by_lhs_[x]) chain(n, from, rules_[r].rhs, 0, rules_[r].rhs.size(), to);
      return;
    }
    // one NFA state per member of the component, private to this instance
    std::map<int, int> st;
    for (int a : info_.scc_members[c]) st[a] = n.add();
    if (kind == 2) {  // right-linear: state of A = "an A is about to start"; whoever ends, ends the instance
      n.eps[from].push_back(st[x]);
      for (int a : info_.scc_members[c])
        for (int r : by_lhs_[a]) {
          const std::vector<int>& rhs = rules_[r].rhs;
          const bool tail = !rhs.empty() && rhs.back() >= 0 && info_.scc_of[rhs.back()] == c;
          if (tail) chain(n, st[a], rhs, 0, rhs.size() - 1, st[rhs.back()]);
          else chain(n, st[a], rhs, 0, rhs.size(), to);
        }
    } else {  // left-linear: state of A = "an A has just ended"
      n.eps[st[x]].push_back(to);
      for (int a : info_.scc_members[c])
        for (int r : by_lhs_[a]) {
          const std::vector<int>& rhs = rules_[r].rhs;
          const bool head = !rhs.empty() && rhs.front() >= 0 && info_.scc_of[rhs.front()] == c;
          if (head) chain(n, st[rhs.front()], rhs, 1, rhs.size(), st[a]);
          else chain(n, from, rhs, 0, rhs.size(), st[a]);
        }
    }
  }

  // ---- subset construction over the byte equivalence classes, then Moore minimisation
  bool determinise(const Nfa& n, int start, int final_state, OneDfa& out) {
    const size_t C = classes_.size();
    std::vector<std::vector<char>> has(C);  // has[c][e]: class c contains the bytes of equivalence class e
    auto closure = [&](std::vector<int>& set) {
      std::vector<int> work = set;
      std::vector<char> in(n.eps.size(), 0);
      for (int s : set) in[s] = 1;
      while (!work.empty()) {
        const int s = work.back();
        work.pop_back();
        for (int t : n.eps[s])
          if (!in[t]) in[t] = 1, set.push_back(t), work.push_back(t);
      }
      std::sort(set.begin(), set.end());
    };
    std::map<std::vector<int>, int> ids;
    std::vector<std::vector<int>> sets;
    std::vector<int> first{start};
    closure(first);
    ids[first] = 0;
    sets.push_back(first);
    std::vector<int> trans;
    for (size_t q = 0; q < sets.size(); ++q) {
      trans.resize((q + 1) * n_eq_, -1);
      for (uint32_t e = 0; e < n_eq_; ++e) {
        const uint32_t byte = rep_[e];
        std::vector<int> next;
        for (int s : sets[q])
          for (auto& ed : n.edge[s]) {
            const int c = ed.first;
            if ((classes_[c][byte >> 5] >> (byte & 31)) & 1u) next.push_back(ed.second);
          }
        if (next.empty()) continue;
        std::sort(next.begin(), next.end());
        next.erase(std::unique(next.begin(), next.end()), next.end());
        closure(next);
        auto it = ids.find(next);
        if (it == ids.end()) {
          if (sets.size() >= DFA_STATE_CAP) return false;
          it = ids.emplace(next, (int)sets.size()).first;
          sets.push_back(next);
        }
        trans[q * n_eq_ + e] = it->second;
      }
    }
    (void)has;
    const size_t S = sets.size();
    std::vector<char> acc(S, 0);
    for (size_t q = 0; q < S; ++q) acc[q] = std::binary_search(sets[q].begin(), sets[q].end(), final_state);
    // Moore: split blocks until every block's members agree on the block of every successor
    std::vector<int> block(S);
    for (size_t q = 0; q < S; ++q) block[q] = acc[q];
    for (size_t n_blocks = 0;;) {
      std::map<std::vector<int>, int> sig_ids;
      std::vector<int> nb(S);
      for (size_t q = 0; q < S; ++q) {
        std::vector<int> sig(n_eq_ + 1);
        sig[0] = block[q];
        for (uint32_t e = 0; e < n_eq_; ++e) sig[e + 1] = trans[q * n_eq_ + e] < 0 ? -1 : block[trans[q * n_eq_ + e]];
        auto it = sig_ids.find(sig);
        if (it == sig_ids.end()) it = sig_ids.emplace(std::move(sig), (int)sig_ids.size()).first;
        nb[q] = it->second;
      }
      block.swap(nb);
      if (sig_ids.size() == n_blocks) break;
      n_blocks = sig_ids.size();
    }
    // number the blocks from the start state's, in order of discovery
    std::vector<int> new_id(S, -1), order;
    std::vector<int> block_id(S, -1);  // block -> new id
    auto take = [&](int q) {
      if (block_id[block[q]] < 0) block_id[block[q]] = (int)order.size(), order.push_back(q);
    };
    take(0);
    for (size_t i = 0; i < order.size(); ++i)
      for (uint32_t e = 0; e < n_eq_; ++e)
        if (trans[(size_t)order[i] * n_eq_ + e] >= 0) take(trans[(size_t)order[i] * n_eq_ + e]);
    out.n_states = (uint32_t)order.size();
    out.trans.assign((size_t)out.n_states * n_eq_, -1);
    out.accepting.assign(out.n_states, 0);
    for (size_t i = 0; i < order.size(); ++i) {
      out.accepting[i] = acc[order[i]];
      for (uint32_t e = 0; e < n_eq_; ++e) {
        const int t = trans[(size_t)order[i] * n_eq_ + e];
        out.trans[i * n_eq_ + e] = t < 0 ? -1 : block_id[block[t]];
      }
    }
    return true;
  }
};

}  // namespace

// ------------------------------------------------------------------------------------ tables

void compile_grammar(const char* text, size_t len, const std::string& start, HostTables& out, bool dfa_terminals) {
  GrammarBuilder b;
  int aug = b.nt("$");
  b.defined[aug] = 1;
  {
    Lexer lx(text, len);
    Parser ps(lx.run(), b);
    ps.run();
  }
  for (size_t i = 0; i < b.names.size(); ++i)
    if (!b.defined[i]) throw CompileError{FMT_ERR_UNDEFINED_SYMBOL, "undefined symbol '" + b.names[i] + "'"};
  int start_id = b.lookup(start);
  if (start_id < 0) throw CompileError{FMT_ERR_UNDEFINED_SYMBOL, "start rule '" + start + "' is not defined"};
  b.prods.insert(b.prods.begin(), Production{aug, {start_id}});

  const size_t n_all = b.names.size();
  // productive non-terminals
  std::vector<char> productive(n_all, 0);
  for (bool again = true; again;) {
    again = false;
    for (auto& p : b.prods) {
      if (productive[p.lhs]) continue;
      bool ok = true;
      for (int s : p.rhs) ok = ok && (s < 0 || productive[s]);
      if (ok) productive[p.lhs] = 1, again = true;
    }
  }
  if (!productive[aug]) throw CompileError{FMT_ERR_EMPTY_LANGUAGE, "the start rule derives no string"};
  std::vector<Production> kept;
  for (auto& p : b.prods) {
    bool ok = productive[p.lhs];
    for (int s : p.rhs) ok = ok && (s < 0 || productive[s]);
    if (ok) kept.push_back(p);
  }
  // reachable from the augmented start
  std::vector<char> reach(n_all, 0);
  reach[aug] = 1;
  for (bool again = true; again;) {
    again = false;
    for (auto& p : kept)
      if (reach[p.lhs])
        for (int s : p.rhs)
          if (s >= 0 && !reach[s]) reach[s] = 1, again = true;
  }
  std::vector<Production> rules;
  for (auto& p : kept)
    if (reach[p.lhs]) rules.push_back(p);
  // nullable
  std::vector<char> nullable(n_all, 0);
  for (bool again = true; again;) {
    again = false;
    for (auto& p : rules) {
      if (nullable[p.lhs]) continue;
      bool ok = true;
      for (int s : p.rhs) ok = ok && (s >= 0 && nullable[s]);
      if (ok) nullable[p.lhs] = 1, again = true;
    }
  }
  // bytes are equivalent when every byte class of the grammar contains both or neither
  out.eq_of_byte.assign(256, 0);
  {
    std::vector<char> used(b.classes.size(), 0);
    for (auto& p : rules)
      for (int s : p.rhs)
        if (s < 0) used[~s] = 1;
    std::map<std::vector<uint8_t>, uint32_t> seen;
    for (int byte = 0; byte < 256; ++byte) {
      std::vector<uint8_t> member;
      for (size_t c = 0; c < b.classes.size(); ++c)
        if (used[c]) member.push_back((b.classes[c][byte >> 5] >> (byte & 31)) & 1u);
      auto it = seen.find(member);
      if (it == seen.end()) it = seen.emplace(member, (uint32_t)seen.size()).first;
      out.eq_of_byte[byte] = (uint8_t)it->second;
    }
    out.n_eq = (uint32_t)seen.size();
  }
  // regular non-terminals used from non-regular rules become automata (see DfaBuilder)
  std::vector<OneDfa> dfas;
  std::vector<int> dfa_of(n_all, -1);
  if (dfa_terminals) {
    DfaBuilder db(rules, n_all, b.classes, out.eq_of_byte, out.n_eq);
    const RegularInfo& ri = db.info();
    std::vector<char> wanted(n_all, 0);
    for (auto& p : rules)
      if (p.lhs == aug || !ri.regular[p.lhs])
        for (int s : p.rhs)
          if (s >= 0 && s != aug && ri.regular[s]) wanted[s] = 1;
    size_t total_states = 0;
    for (size_t x = 0; x < n_all; ++x) {
      if (!wanted[x]) continue;
      OneDfa one;
      if (!db.build((int)x, one)) continue;                        // too large: stays a set of rules
      if (total_states + one.n_states > 16000) continue;           // (state numbers have 14 bits)
      total_states += one.n_states;
      dfa_of[x] = (int)dfas.size();
      dfas.push_back(std::move(one));
    }
    if (!dfas.empty()) {  // their rules go, and with them whatever only they used
      std::vector<Production> left;
      for (auto& p : rules)
        if (dfa_of[p.lhs] < 0) left.push_back(p);
      std::vector<char> r2(n_all, 0);
      r2[aug] = 1;
      for (bool again = true; again;) {
        again = false;
        for (auto& p : left)
          if (r2[p.lhs])
            for (int s : p.rhs)
              if (s >= 0 && !r2[s]) r2[s] = 1, again = dfa_of[s] < 0 || again;
      }
      rules.clear();
      for (auto& p : left)
        if (r2[p.lhs]) rules.push_back(p);
      for (size_t x = 0; x < n_all; ++x)
        if (dfa_of[x] >= 0 && !r2[x]) dfa_of[x] = -2;  // (built but no longer used: cannot happen, kept for safety)
    }
  }
  // renumber non-terminals ($ = 0) and byte classes (only those still used)
  std::vector<int> nt_new(n_all, -1);
  int N = 0;
  nt_new[aug] = N++;
  for (auto& p : rules)
    if (nt_new[p.lhs] < 0) nt_new[p.lhs] = N++;
  for (auto& p : rules)
    for (int s : p.rhs)
      if (s >= 0 && nt_new[s] < 0) nt_new[s] = N++;  // (non-terminals that are automata have no rules)
  std::vector<int> cls_new(b.classes.size(), -1);
  int C = 0;
  for (auto& p : rules)
    for (int s : p.rhs)
      if (s < 0 && cls_new[~s] < 0) cls_new[~s] = C++;
  // empty productions are dropped: their effect lives in the nullable flags
  std::vector<Production> solid;
  for (auto& p : rules)
    if (!p.rhs.empty()) solid.push_back(p);
  size_t D = 0;
  for (auto& p : solid) D += p.rhs.size() + 1;
  // after the rule positions: one item id per automaton state, then one "done" id per automaton
  const size_t D_rules = D;
  size_t S_total = 0;
  std::vector<int> used_dfas;
  for (size_t x = 0; x < n_all; ++x)
    if (dfa_of[x] >= 0) used_dfas.push_back((int)x);
  for (int x : used_dfas) S_total += dfas[dfa_of[x]].n_states;
  D += S_total + used_dfas.size();
  if (D > 65535 || N > (int)MAX_NONTERMINALS || C > 65535)
    throw CompileError{FMT_ERR_CAPACITY, "grammar too large: more than 65535 dotted rules or classes, or 4096 non-terminals"};

  out.N = (uint32_t)N;
  out.P = (uint32_t)solid.size();
  out.D = (uint32_t)D;
  out.C = (uint32_t)C;
  out.Nw = ((uint32_t)N + 31) / 32;
  out.nullable.assign(N, 0);
  out.nt_names.assign(N, "");
  out.n_nullable = 0;
  for (size_t i = 0; i < n_all; ++i)
    if (nt_new[i] >= 0) {
      out.nullable[nt_new[i]] = (uint8_t)nullable[i];
      out.nt_names[nt_new[i]] = b.names[i];
      out.n_nullable += nullable[i] ? 1 : 0;
    }
  out.start_nullable = nullable[start_id] != 0;
  out.class_bits.assign((size_t)std::max(C, 1) * 8, 0);
  for (size_t c = 0; c < b.classes.size(); ++c)
    if (cls_new[c] >= 0)
      for (int w = 0; w < 8; ++w) out.class_bits[(size_t)cls_new[c] * 8 + w] = b.classes[c][w];

  out.info.assign(D, 0);
  out.lhs.assign(D, 0);
  out.skip.assign(D, 0);
  std::vector<std::vector<uint32_t>> first_item(N);  // start item of each rule, per non-terminal
  // the automata: item id dfa_first + g is "state g" (all automata's states numbered in a row), the ids
  // after them are the completed items of the non-terminals they stand for
  out.dfa_first = (uint32_t)D_rules;
  out.dfa_states = (uint32_t)S_total;
  out.dfa_trans.assign(S_total * out.n_eq, 0xFFFFu);
  out.dfa_done.assign(S_total, 0);
  out.dfa_scan.assign(S_total * 8, 0);
  out.dfa_accept.assign(S_total, 0);
  out.dfa_nt.clear();
  out.dfa_start.clear();
  {
    uint32_t g0 = 0;
    for (size_t j = 0; j < used_dfas.size(); ++j) {
      const OneDfa& a = dfas[dfa_of[used_dfas[j]]];
      const int L = nt_new[used_dfas[j]];
      const uint32_t done_id = (uint32_t)(D_rules + S_total + j);
      out.dfa_nt.push_back((uint32_t)L);
      out.dfa_start.push_back(g0);
      first_item[L].push_back(out.dfa_first + g0);
      out.info[done_id] = (KIND_END << INFO_KIND_SHIFT) | (uint32_t)L;
      out.lhs[done_id] = (uint16_t)L;
      for (uint32_t q = 0; q < a.n_states; ++q) {
        const uint32_t g = g0 + q;
        out.info[out.dfa_first + g] = (KIND_DFA << INFO_KIND_SHIFT) | g;
        out.lhs[out.dfa_first + g] = (uint16_t)L;
        out.dfa_done[g] = (uint16_t)done_id;
        out.dfa_accept[g] = (uint8_t)a.accepting[q];
        for (uint32_t e = 0; e < out.n_eq; ++e) {
          const int t = a.trans[(size_t)q * out.n_eq + e];
          if (t < 0) continue;
          bool alive = false;  // a state nothing leaves is never made an item: a finished automaton is dropped at once
          for (uint32_t e2 = 0; e2 < out.n_eq; ++e2) alive = alive || a.trans[(size_t)t * out.n_eq + e2] >= 0;
          out.dfa_trans[(size_t)g * out.n_eq + e] =
              (uint16_t)((g0 + (uint32_t)t) | (alive ? 0x4000u : 0u) | (a.accepting[t] ? 0x8000u : 0u));
          for (int byte = 0; byte < 256; ++byte)
            if (out.eq_of_byte[byte] == e) out.dfa_scan[(size_t)g * 8 + (byte >> 5)] |= 1u << (byte & 31);
        }
      }
      g0 += a.n_states;
    }
  }
  uint32_t d = 0;
  for (auto& p : solid) {  // solid[0] is $ -> start, so items 0 and 1 are the start and accept items
    int L = nt_new[p.lhs];
    first_item[L].push_back(d);
    for (size_t k = 0; k <= p.rhs.size(); ++k, ++d) {
      out.lhs[d] = (uint16_t)L;
      if (k == p.rhs.size()) {
        out.info[d] = (KIND_END << INFO_KIND_SHIFT) | (uint32_t)L;
      } else if (p.rhs[k] < 0) {
        out.info[d] = (KIND_TERM << INFO_KIND_SHIFT) | (uint32_t)cls_new[~p.rhs[k]];
      } else {
        uint32_t y = (uint32_t)nt_new[p.rhs[k]];
        out.info[d] = (KIND_NT << INFO_KIND_SHIFT) | y | (out.nullable[y] ? INFO_NULLABLE : 0u);
      }
    }
  }
  for (uint32_t i = (uint32_t)D_rules; i-- > 0;)
    if ((out.info[i] >> INFO_KIND_SHIFT) == KIND_NT && (out.info[i] & INFO_NULLABLE))
      out.skip[i] = (uint8_t)std::min<uint32_t>(255u, 1u + out.skip[i + 1]);
  for (uint32_t i = 0; i < (uint32_t)D; ++i) out.info[i] |= (uint32_t)out.skip[i] << INFO_SKIP_SHIFT;
  // direct items: the start item of every rule plus the items reached by moving the dot over
  // leading nullable non-terminals; completed items are left out (their effect is the parent's skip)
  out.direct_off.assign(N + 1, 0);
  out.direct_items.clear();
  for (int y = 0; y < N; ++y) {
    out.direct_off[y] = (uint32_t)out.direct_items.size();
    for (uint32_t s : first_item[y])
      for (uint32_t j = 0; j <= out.skip[s]; ++j)
        if ((out.info[s + j] >> INFO_KIND_SHIFT) != KIND_END) out.direct_items.push_back((uint16_t)(s + j));
  }
  out.direct_off[N] = (uint32_t)out.direct_items.size();
  if (out.direct_items.empty()) out.direct_items.push_back(0);
  // closure of "predicting Y also predicts Z"
  out.nt_closure.assign((size_t)N * out.Nw, 0);
  for (int y = 0; y < N; ++y) {
    uint32_t* row = &out.nt_closure[(size_t)y * out.Nw];
    std::vector<int> work{y};
    row[y >> 5] |= 1u << (y & 31);
    while (!work.empty()) {
      int z = work.back();
      work.pop_back();
      for (uint32_t k = out.direct_off[z]; k < out.direct_off[z + 1]; ++k) {
        uint32_t inf = out.info[out.direct_items[k]];
        if ((inf >> INFO_KIND_SHIFT) == KIND_NT) {
          uint32_t w = inf & INFO_ARG_MASK;
          if (!((row[w >> 5] >> (w & 31)) & 1u)) row[w >> 5] |= 1u << (w & 31), work.push_back((int)w);
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------ trie

void build_trie(const uint8_t* bytes, const uint64_t* offs, uint32_t V, int32_t eos, HostTables& out) {
  out.V = V;
  out.Wm = (V + 31) / 32;
  out.eos = eos;
  out.vocab_off.assign((size_t)V + 1, 0);
  out.n_empty = 0;
  for (uint32_t t = 0; t < V; ++t)
    if (offs[t + 1] < offs[t]) throw CompileError{FMT_ERR_INVALID_ARG, "vocab_offsets must not decrease"};
  uint64_t total = offs[V] - offs[0];
  if (total > 0xFFFFFFF0ull) throw CompileError{FMT_ERR_CAPACITY, "vocabulary bytes exceed 4 GiB"};
  out.vocab_bytes.assign(bytes + offs[0], bytes + offs[V]);
  if (out.vocab_bytes.empty()) out.vocab_bytes.push_back(0);
  std::vector<uint32_t> order;
  order.reserve(V);
  for (uint32_t t = 0; t < V; ++t) {
    uint64_t l = offs[t + 1] - offs[t];
    if (l > MAX_TOKEN_BYTES)
      throw CompileError{FMT_ERR_CAPACITY, "token " + std::to_string(t) + " is longer than 32 bytes"};
    out.vocab_off[t] = (uint32_t)(offs[t] - offs[0]);
    if (l == 0) ++out.n_empty;
    else order.push_back(t);
  }
  out.vocab_off[V] = (uint32_t)total;
  const uint8_t* base = out.vocab_bytes.data();
  auto tok_len = [&](uint32_t t) { return out.vocab_off[t + 1] - out.vocab_off[t]; };
  auto tok_ptr = [&](uint32_t t) { return base + out.vocab_off[t]; };
  std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
    uint32_t la = tok_len(a), lb = tok_len(b);
    int c = memcmp(tok_ptr(a), tok_ptr(b), std::min(la, lb));
    if (c != 0) return c < 0;
    if (la != lb) return la < lb;
    return a < b;
  });
  // breadth-first construction over ranges of the sorted token list
  struct Range {
    uint32_t lo, hi, depth;
  };
  out.child_off.clear();
  out.node_byte.clear();
  out.parent.clear();
  out.node_depth.clear();
  out.tok_off.clear();
  out.tok_ids.clear();
  std::vector<Range> nodes;
  nodes.push_back({0, (uint32_t)order.size(), 0});
  out.node_byte.push_back(0);
  out.parent.push_back(0);
  out.node_depth.push_back(0);
  out.depth = 0;
  for (size_t n = 0; n < nodes.size(); ++n) {
    Range r = nodes[n];
    out.child_off.push_back((uint32_t)nodes.size());
    out.tok_off.push_back((uint32_t)out.tok_ids.size());
    uint32_t i = r.lo;
    while (i < r.hi && tok_len(order[i]) == r.depth) out.tok_ids.push_back(order[i++]);  // tokens ending here
    while (i < r.hi) {
      uint8_t c = tok_ptr(order[i])[r.depth];
      uint32_t j = i;
      while (j < r.hi && tok_ptr(order[j])[r.depth] == c) ++j;
      nodes.push_back({i, j, r.depth + 1});
      out.node_byte.push_back(c);
      out.parent.push_back((uint32_t)n);
      out.node_depth.push_back((uint8_t)(r.depth + 1));
      out.depth = std::max(out.depth, r.depth + 1);
      i = j;
    }
  }
  out.T = (uint32_t)nodes.size();
  out.child_off.push_back(out.T);
  out.tok_off.push_back((uint32_t)out.tok_ids.size());
  if (out.tok_ids.empty()) out.tok_ids.push_back(0);
  // breadth-first numbering makes every depth a contiguous range of nodes
  out.lvl_off.assign(out.depth + 2, out.T);
  out.lvl_off[0] = 0;
  for (uint32_t n = out.T; n-- > 0;) out.lvl_off[out.node_depth[n]] = n;
  out.lvl_off[out.depth + 1] = out.T;
  for (uint32_t L = out.depth; L >= 1; --L)
    if (out.lvl_off[L] > out.lvl_off[L + 1]) out.lvl_off[L] = out.lvl_off[L + 1];
  out.tok_node.assign(V, 0xFFFFFFFFu);
  for (uint32_t n = 0; n < out.T; ++n)
    for (uint32_t i = out.tok_off[n]; i < out.tok_off[n + 1] && i < (uint32_t)order.size(); ++i) out.tok_node[out.tok_ids[i]] = n;
}

}  // namespace fmt
