// TEST INFRASTRUCTURE — not part of the product path.
//
// A plain, slow CPU oracle for grammar-constrained vocabulary masking, written from the
// paper "Earley-Driven Dynamic Pruning for Efficient Structured Decoding" (Section 3.2:
// Earley sets, predict / scan / complete; Section 3.3: the logits mask; Section 4.2:
// ZapFormat pruning; Section 4.5: useless-rule removal).  It shares no code with the CUDA
// library: own grammar-text parser, own grammar reduction, own recognizer.
//
// What it computes (the definition the mask follows, Section 3.3 / Section 4.1):
//   mask[t] = 1  <=>  bytes(t) is non-empty and  w . bytes(t)  is a viable prefix of L(G)
//   mask[eos] = 1 <=> w is a sentence of L(G)
// where w is the byte string advanced so far.  With every non-terminal productive and
// reachable (Section 4.5), "viable prefix" equals "every Earley set stays non-empty".
//
// Two recognizers live here:
//   * Full     - textbook Earley with the whole chart S[0..n] kept (Section 3.2).  Each
//                vocabulary token is checked on its own by building the token's sets on top
//                of the shared prefix chart.  This is THE oracle.
//   * Pruned   - the same recognizer followed, after each byte, by a Compact step in the
//                reading of Figure 3's caption: completed items are dropped once their set
//                is finished, and an item of an earlier set survives only if a chain of
//                Complete references from the last set reaches it.  Used for the invariant
//                "pruned and unpruned charts accept the same tokens" and for the worked
//                example of Section 1.  Pinned by that example only; chart contents beyond
//                it are "parity unpinned" (they never reach the mask).
//
// Build: g++ -O2 -std=c++17 -fopenmp -shared -fPIC earley_oracle.cpp -o liboracle.so
#include <algorithm>
#include <array>
#include <bitset>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <functional>
#include <map>
#include <memory>
#include <set>
#include <stdexcept>
#include <string>
#include <unordered_set>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum Status { OK = 0, BAD_ARG = 1, SYNTAX = 2, UNDEFINED_SYMBOL = 3, EMPTY_LANGUAGE = 4 };

struct GrammarError {
  int code;
  std::string msg;
};

using ByteClass = std::bitset<256>;

struct Sym {
  bool terminal;
  int id;  // terminal: index into classes; non-terminal: index into names
};

struct Rule {
  int lhs;
  std::vector<Sym> rhs;
};

// ------------------------------------------------------------------ grammar text -> AST

struct Node {
  enum Kind { LITERAL, CLASS, NAME, SEQ, ALT, STAR, PLUS, OPT } kind;
  std::string text;        // LITERAL bytes / NAME
  ByteClass cls;           // CLASS
  std::vector<Node> kids;  // SEQ / ALT / postfix operand
};

class TextParser {
 public:
  TextParser(const char* s, size_t n) : s_(s), n_(n) {}

  std::vector<std::pair<std::string, Node>> parse() {
    std::vector<std::pair<std::string, Node>> out;
    skip();
    while (i_ < n_) {
      std::string name = ident();
      if (name.empty()) fail("expected a rule name");
      skip();
      if (!eat("::=")) fail("expected ::= after " + name);
      Node body = alternation();
      out.emplace_back(name, std::move(body));
      skip();
    }
    return out;
  }

 private:
  const char* s_;
  size_t n_;
  size_t i_ = 0;

  [[noreturn]] void fail(const std::string& m) {
    throw GrammarError{SYNTAX, m + " at offset " + std::to_string(i_)};
  }
  void skip() {
    while (i_ < n_) {
      char c = s_[i_];
      if (c == ' ' || c == '\t' || c == '\n' || c == '\r') {
        ++i_;
      } else if (c == '#') {
        while (i_ < n_ && s_[i_] != '\n') ++i_;
      } else {
        break;
      }
    }
  }
  bool eat(const char* t) {
    size_t l = strlen(t);
    if (i_ + l <= n_ && memcmp(s_ + i_, t, l) == 0) {
      i_ += l;
      return true;
    }
    return false;
  }
  static bool ident_start(char c) { return (c >= 'a' && c <= 'z') || (c >= 'A' && c <= 'Z') || c == '_'; }
  static bool ident_char(char c) { return ident_start(c) || (c >= '0' && c <= '9') || c == '-'; }
  std::string ident() {
    size_t j = i_;
    if (j < n_ && ident_start(s_[j])) {
      ++j;
      while (j < n_ && ident_char(s_[j])) ++j;
    }
    std::string r(s_ + i_, j - i_);
    i_ = j;
    return r;
  }
  // does a new rule (`name ::=`) start here?
  bool at_rule_start() {
    size_t save = i_;
    std::string nm = ident();
    bool yes = false;
    if (!nm.empty()) {
      skip();
      yes = (i_ + 3 <= n_ && memcmp(s_ + i_, "::=", 3) == 0);
    }
    i_ = save;
    return yes;
  }
  int hexval(char c) {
    if (c >= '0' && c <= '9') return c - '0';
    if (c >= 'a' && c <= 'f') return c - 'a' + 10;
    if (c >= 'A' && c <= 'F') return c - 'A' + 10;
    fail("bad hex digit");
  }
  unsigned char escape() {  // after the backslash
    if (i_ >= n_) fail("dangling backslash");
    char c = s_[i_++];
    switch (c) {
      case 'n': return '\n';
      case 'r': return '\r';
      case 't': return '\t';
      case 'x': {
        if (i_ + 2 > n_) fail("short \\x escape");
        int v = hexval(s_[i_]) * 16 + hexval(s_[i_ + 1]);
        i_ += 2;
        return (unsigned char)v;
      }
      default: return (unsigned char)c;  // \\ \" \] \- \^ and any other char stand for themselves
    }
  }
  Node alternation() {
    Node alt{Node::ALT};
    alt.kids.push_back(sequence());
    skip();
    while (i_ < n_ && s_[i_] == '|') {
      ++i_;
      alt.kids.push_back(sequence());
      skip();
    }
    if (alt.kids.size() == 1) return alt.kids[0];
    return alt;
  }
  Node sequence() {
    Node seq{Node::SEQ};
    for (;;) {
      skip();
      if (i_ >= n_) break;
      char c = s_[i_];
      if (c == '|' || c == ')') break;
      if (ident_start(c) && at_rule_start()) break;
      seq.kids.push_back(postfix());
    }
    return seq;
  }
  Node postfix() {
    Node a = atom();
    for (;;) {
      skip();
      if (i_ >= n_) break;
      char c = s_[i_];
      Node::Kind k;
      if (c == '*') k = Node::STAR;
      else if (c == '+') k = Node::PLUS;
      else if (c == '?') k = Node::OPT;
      else break;
      ++i_;
      Node p{k};
      p.kids.push_back(std::move(a));
      a = std::move(p);
    }
    return a;
  }
  Node atom() {
    char c = s_[i_];
    if (c == '"') {
      ++i_;
      Node lit{Node::LITERAL};
      for (;;) {
        if (i_ >= n_) fail("unterminated literal");
        char d = s_[i_++];
        if (d == '"') break;
        if (d == '\\') lit.text.push_back((char)escape());
        else lit.text.push_back(d);
      }
      return lit;
    }
    if (c == '[') {
      ++i_;
      Node cl{Node::CLASS};
      bool neg = false;
      if (i_ < n_ && s_[i_] == '^') {
        neg = true;
        ++i_;
      }
      for (;;) {
        if (i_ >= n_) fail("unterminated class");
        char d = s_[i_++];
        if (d == ']') break;
        unsigned char lo = (d == '\\') ? escape() : (unsigned char)d;
        unsigned char hi = lo;
        if (i_ + 1 < n_ && s_[i_] == '-' && s_[i_ + 1] != ']') {
          ++i_;
          char e = s_[i_++];
          hi = (e == '\\') ? escape() : (unsigned char)e;
          if (hi < lo) fail("reversed range in class");
        }
        for (int b = lo; b <= hi; ++b) cl.cls.set(b);
      }
      if (neg) cl.cls.flip();
      if (cl.cls.none()) fail("empty byte class");
      return cl;
    }
    if (c == '(') {
      ++i_;
      Node inner = alternation();
      skip();
      if (i_ >= n_ || s_[i_] != ')') fail("expected )");
      ++i_;
      return inner;
    }
    if (ident_start(c)) {
      Node nm{Node::NAME};
      nm.text = ident();
      return nm;
    }
    fail(std::string("unexpected character '") + c + "'");
  }
};

// ------------------------------------------------------------------ AST -> reduced rule list

struct Grammar {
  std::vector<std::string> names;  // non-terminal names; index 0 is the augmented start $
  std::vector<ByteClass> classes;
  std::vector<Rule> rules;         // rules[0] is  $ -> start
  std::vector<std::vector<int>> rules_of;

  std::string sym_text(const Sym& s) const {
    if (!s.terminal) return names[s.id];
    const ByteClass& c = classes[s.id];
    if (c.count() == 1) {
      for (int b = 0; b < 256; ++b)
        if (c.test(b)) {
          char buf[8];
          if (b > 0x20 && b < 0x7f) snprintf(buf, sizeof buf, "%c", b);
          else snprintf(buf, sizeof buf, "x%02x", b);
          return buf;
        }
    }
    std::string r = "[";
    for (int b = 0; b < 256; ++b)
      if (c.test(b)) {
        char buf[8];
        snprintf(buf, sizeof buf, "%02x", b);
        r += buf;
      }
    return r + "]";
  }
};

class Builder {
 public:
  Grammar build(const char* text, size_t len, const std::string& start) {
    TextParser tp(text, len);
    auto parsed = tp.parse();
    if (parsed.empty()) throw GrammarError{SYNTAX, "no rules"};
    g_.names.push_back("$");
    for (auto& pr : parsed) {
      if (!index_.count(pr.first)) {
        index_[pr.first] = (int)g_.names.size();
        g_.names.push_back(pr.first);
      }
    }
    if (!index_.count(start)) throw GrammarError{UNDEFINED_SYMBOL, "start rule '" + start + "' is not defined"};
    g_.rules.push_back(Rule{0, {Sym{false, index_[start]}}});
    for (auto& pr : parsed) add_alternatives(index_[pr.first], pr.second);
    reduce();
    g_.rules_of.assign(g_.names.size(), {});
    for (size_t r = 0; r < g_.rules.size(); ++r) g_.rules_of[g_.rules[r].lhs].push_back((int)r);
    return std::move(g_);
  }

 private:
  Grammar g_;
  std::map<std::string, int> index_;
  int fresh_ = 0;

  int fresh_nt(const std::string base) {
    std::string nm = base + "%" + std::to_string(++fresh_);
    g_.names.push_back(nm);
    return (int)g_.names.size() - 1;
  }
  void add_alternatives(int lhs, const Node& n) {
    if (n.kind == Node::ALT) {
      for (auto& k : n.kids) add_alternatives(lhs, k);
      return;
    }
    Rule r{lhs, {}};
    append(r.rhs, n, g_.names[lhs]);
    g_.rules.push_back(std::move(r));
  }
  // append the symbols of node n to rhs, introducing fresh non-terminals where needed
  void append(std::vector<Sym>& rhs, const Node& n, const std::string ctx) {
    switch (n.kind) {
      case Node::LITERAL:
        for (unsigned char ch : n.text) {
          ByteClass c;
          c.set(ch);
          g_.classes.push_back(c);
          rhs.push_back(Sym{true, (int)g_.classes.size() - 1});
        }
        break;
      case Node::CLASS:
        g_.classes.push_back(n.cls);
        rhs.push_back(Sym{true, (int)g_.classes.size() - 1});
        break;
      case Node::NAME: {
        auto it = index_.find(n.text);
        if (it == index_.end()) throw GrammarError{UNDEFINED_SYMBOL, "undefined symbol '" + n.text + "'"};
        rhs.push_back(Sym{false, it->second});
        break;
      }
      case Node::SEQ:
        for (auto& k : n.kids) append(rhs, k, ctx);
        break;
      case Node::ALT: {
        int x = fresh_nt(ctx);
        add_alternatives(x, n);
        rhs.push_back(Sym{false, x});
        break;
      }
      case Node::OPT: {  // X -> inner | empty
        int x = fresh_nt(ctx);
        add_alternatives(x, n.kids[0]);
        g_.rules.push_back(Rule{x, {}});
        rhs.push_back(Sym{false, x});
        break;
      }
      case Node::STAR: {  // X -> inner X | empty   (right recursive here; the direction does not change L(G))
        int x = fresh_nt(ctx);
        Rule r{x, {}};
        append(r.rhs, n.kids[0], ctx);
        r.rhs.push_back(Sym{false, x});
        g_.rules.push_back(std::move(r));
        g_.rules.push_back(Rule{x, {}});
        rhs.push_back(Sym{false, x});
        break;
      }
      case Node::PLUS: {  // X -> inner X | inner
        int x = fresh_nt(ctx);
        Rule r1{x, {}}, r2{x, {}};
        append(r1.rhs, n.kids[0], ctx);
        r2.rhs = r1.rhs;
        r1.rhs.push_back(Sym{false, x});
        g_.rules.push_back(std::move(r1));
        g_.rules.push_back(std::move(r2));
        rhs.push_back(Sym{false, x});
        break;
      }
    }
  }
  // Section 4.5: drop rules that cannot take part in a derivation of a sentence.
  void reduce() {
    size_t N = g_.names.size();
    std::vector<char> productive(N, 0);
    bool changed = true;
    while (changed) {
      changed = false;
      for (auto& r : g_.rules) {
        if (productive[r.lhs]) continue;
        bool all = true;
        for (auto& s : r.rhs)
          if (!s.terminal && !productive[s.id]) {
            all = false;
            break;
          }
        if (all) {
          productive[r.lhs] = 1;
          changed = true;
        }
      }
    }
    if (!productive[0]) throw GrammarError{EMPTY_LANGUAGE, "the start rule derives no string"};
    std::vector<Rule> kept;
    for (auto& r : g_.rules) {
      bool all = productive[r.lhs];
      for (auto& s : r.rhs)
        if (!s.terminal && !productive[s.id]) all = false;
      if (all) kept.push_back(r);
    }
    std::vector<char> reach(N, 0);
    reach[0] = 1;
    changed = true;
    while (changed) {
      changed = false;
      for (auto& r : kept)
        if (reach[r.lhs])
          for (auto& s : r.rhs)
            if (!s.terminal && !reach[s.id]) {
              reach[s.id] = 1;
              changed = true;
            }
    }
    std::vector<Rule> kept2;
    for (auto& r : kept)
      if (reach[r.lhs]) kept2.push_back(r);
    g_.rules = std::move(kept2);  // rules[0] is still the augmented rule (it was first and is kept)
  }
};

// ------------------------------------------------------------------ Earley items and sets

struct Item {
  int rule, dot, origin;
  bool operator==(const Item& o) const { return rule == o.rule && dot == o.dot && origin == o.origin; }
  bool operator<(const Item& o) const {
    if (rule != o.rule) return rule < o.rule;
    if (dot != o.dot) return dot < o.dot;
    return origin < o.origin;
  }
};

struct ItemSet {  // an Earley set holds every item at most once (Section 3.2)
  std::vector<Item> items;
  std::unordered_set<uint64_t> seen;
  static uint64_t key(const Item& it) {
    return ((uint64_t)(uint32_t)it.rule << 44) ^ ((uint64_t)(uint32_t)it.dot << 32) ^ (uint64_t)(uint32_t)it.origin;
  }
  bool add(const Item& it) {
    if (!seen.insert(key(it)).second) return false;
    items.push_back(it);
    return true;
  }
  void clear() {
    items.clear();
    seen.clear();
  }
  bool empty() const { return items.empty(); }
};

// Predict and Complete on set `cur` (whose index is k) until nothing is added.  `lookup(j)`
// returns set j for j < k.  A naive whole-set fixpoint: rules that derive the empty string
// need no special case because a completion with origin k re-reads set k on the next pass.
template <class Lookup>
void closure(const Grammar& g, ItemSet& cur, int k, Lookup lookup) {
  bool changed = true;
  while (changed) {
    changed = false;
    for (size_t idx = 0; idx < cur.items.size(); ++idx) {
      Item it = cur.items[idx];
      const Rule& r = g.rules[it.rule];
      if (it.dot < (int)r.rhs.size()) {
        const Sym& s = r.rhs[it.dot];
        if (!s.terminal)  // Predict: add every rule of the post-dot non-terminal, starting at k
          for (int q : g.rules_of[s.id])
            if (cur.add(Item{q, 0, k})) changed = true;
      } else {  // Complete: advance every item of set `origin` whose post-dot symbol is this lhs
        int X = r.lhs;
        const std::vector<Item>& from = (it.origin == k) ? cur.items : lookup(it.origin).items;
        size_t n = from.size();  // `from` may be cur.items and grow; later items are met on the next pass
        for (size_t j = 0; j < n; ++j) {
          Item w = (it.origin == k) ? cur.items[j] : from[j];
          const Rule& wr = g.rules[w.rule];
          if (w.dot < (int)wr.rhs.size() && !wr.rhs[w.dot].terminal && wr.rhs[w.dot].id == X)
            if (cur.add(Item{w.rule, w.dot + 1, w.origin})) changed = true;
        }
      }
    }
  }
}

// Scan: items of `from` whose post-dot terminal matches byte b, advanced, go to `to`.
void scan(const Grammar& g, const ItemSet& from, unsigned char b, ItemSet& to) {
  for (const Item& it : from.items) {
    const Rule& r = g.rules[it.rule];
    if (it.dot < (int)r.rhs.size() && r.rhs[it.dot].terminal && g.classes[r.rhs[it.dot].id].test(b))
      to.add(Item{it.rule, it.dot + 1, it.origin});
  }
}

bool has_accept(const ItemSet& s) {  // ($ -> start . , 0)
  for (const Item& it : s.items)
    if (it.rule == 0 && it.dot == 1 && it.origin == 0) return true;
  return false;
}

std::string item_text(const Grammar& g, const Item& it) {
  const Rule& r = g.rules[it.rule];
  std::string s = g.names[r.lhs] + " ->";
  for (size_t i = 0; i <= r.rhs.size(); ++i) {
    if ((int)i == it.dot) s += " .";
    if (i < r.rhs.size()) s += " " + g.sym_text(r.rhs[i]);
  }
  s += " ; " + std::to_string(it.origin);
  return s;
}

struct Vocab {
  std::vector<std::string> tok;
  int eos;
};

// ------------------------------------------------------------------ the two recognizers

struct Seq {
  const Grammar* g;
  bool pruned;
  std::vector<ItemSet> chart;  // Full: S[0..n].  Pruned: the surviving sets, densely renumbered.
  bool accepting = false;
  size_t n_bytes = 0;
  size_t peak_items = 0;

  Seq(const Grammar* gr, bool pr) : g(gr), pruned(pr) {
    chart.emplace_back();
    chart[0].add(Item{0, 0, 0});
    closure(*g, chart[0], 0, [&](int j) -> const ItemSet& { return chart[j]; });
    accepting = has_accept(chart[0]);
    if (pruned) compact();
    track();
  }
  void track() {
    size_t t = 0;
    for (auto& s : chart) t += s.items.size();
    peak_items = std::max(peak_items, t);
  }
  size_t total_items() const {
    size_t t = 0;
    for (auto& s : chart) t += s.items.size();
    return t;
  }

  // Extend a copy-free view of the chart by `bytes`; returns false as soon as a set is empty.
  // `ext` receives the new sets.  Works for both recognizers: in the pruned one the chart's
  // last set plays the role of S[n] and origins index the renumbered sets.
  bool extend(const unsigned char* bytes, size_t n, std::vector<ItemSet>& ext) const {
    int base = (int)chart.size();
    ext.resize(n);
    for (size_t i = 0; i < n; ++i) {
      ext[i].clear();
      const ItemSet& prev = (i == 0) ? chart.back() : ext[i - 1];
      scan(*g, prev, bytes[i], ext[i]);
      if (ext[i].empty()) return false;
      int k = base + (int)i;
      closure(*g, ext[i], k, [&](int j) -> const ItemSet& { return j < base ? chart[j] : ext[j - base]; });
    }
    return true;
  }

  bool advance(const unsigned char* bytes, size_t n) {
    if (!pruned) {
      std::vector<ItemSet> ext;
      if (!extend(bytes, n, ext)) return false;
      for (auto& s : ext) chart.push_back(std::move(s));
      accepting = has_accept(chart.back());
      n_bytes += n;
      track();
      return true;
    }
    // pruned: byte by byte with Compact after each; roll back on rejection
    std::vector<ItemSet> save = chart;
    bool save_acc = accepting;
    for (size_t i = 0; i < n; ++i) {
      ItemSet next;
      scan(*g, chart.back(), bytes[i], next);
      if (next.empty()) {
        chart = std::move(save);
        accepting = save_acc;
        return false;
      }
      int k = (int)chart.size();
      chart.push_back(std::move(next));
      closure(*g, chart[k], k, [&](int j) -> const ItemSet& { return chart[j]; });
      accepting = has_accept(chart[k]);
      compact();
      track();
    }
    n_bytes += n;
    return true;
  }

  // Compact (Section 4.2.3, Figure 3): keep
  //   - in the last set: every item whose dot is not at the end;
  //   - in earlier sets: an item (Y -> mu . A nu, o') of set o only if some kept item with
  //     left-hand side A and origin o exists (a future Complete of that item reads it);
  // drop everything else, drop sets left empty, renumber origins densely.
  void compact() {
    int last = (int)chart.size() - 1;
    std::vector<std::vector<char>> live(chart.size());
    for (size_t k = 0; k < chart.size(); ++k) live[k].assign(chart[k].items.size(), 0);
    std::set<std::pair<int, int>> need;          // (set index, non-terminal)
    std::vector<std::pair<int, int>> work;
    auto raise = [&](int o, int A) {
      if (need.insert({o, A}).second) work.push_back({o, A});
    };
    for (size_t i = 0; i < chart[last].items.size(); ++i) {
      const Item& it = chart[last].items[i];
      const Rule& r = g->rules[it.rule];
      if (it.dot < (int)r.rhs.size()) {
        live[last][i] = 1;
        raise(it.origin, r.lhs);
      }
    }
    while (!work.empty()) {
      auto [o, A] = work.back();
      work.pop_back();
      for (size_t i = 0; i < chart[o].items.size(); ++i) {
        const Item& it = chart[o].items[i];
        const Rule& r = g->rules[it.rule];
        if (it.dot < (int)r.rhs.size() && !r.rhs[it.dot].terminal && r.rhs[it.dot].id == A) {
          if (!live[o][i]) {
            live[o][i] = 1;
            raise(it.origin, r.lhs);
          }
        }
      }
    }
    std::vector<int> renum(chart.size(), -1);
    int m = 0;
    for (size_t k = 0; k < chart.size(); ++k) {
      bool any = false;
      for (char c : live[k]) any = any || c;
      if (any || (int)k == last) renum[k] = m++;
    }
    std::vector<ItemSet> out(m);
    for (size_t k = 0; k < chart.size(); ++k) {
      if (renum[k] < 0) continue;
      std::vector<Item> kept;
      for (size_t i = 0; i < chart[k].items.size(); ++i)
        if (live[k][i]) {
          Item it = chart[k].items[i];
          it.origin = renum[it.origin];
          kept.push_back(it);
        }
      std::sort(kept.begin(), kept.end());
      for (auto& it : kept) out[renum[k]].add(it);
    }
    chart = std::move(out);
  }

  std::string set_text(size_t k) const {
    std::vector<std::string> lines;
    for (auto& it : chart[k].items) lines.push_back(item_text(*g, it));
    std::sort(lines.begin(), lines.end());
    std::string s;
    for (auto& l : lines) s += l + "\n";
    return s;
  }
  // canonical text of the whole (pruned) chart: what a state cache would key on
  std::string key_text() const {
    std::string s = accepting ? "accepting\n" : "not accepting\n";
    for (size_t k = 0; k < chart.size(); ++k) s += "set " + std::to_string(k) + "\n" + set_text(k);
    return s;
  }
};

thread_local std::string g_err;

}  // namespace

// ====================================================================== C interface

extern "C" {

int orc_grammar_new(const char* ebnf, size_t len, const char* start, void** out, char* err, size_t errlen) {
  try {
    Builder b;
    auto* g = new Grammar(b.build(ebnf, len, start));
    *out = g;
    return OK;
  } catch (const GrammarError& e) {
    if (err && errlen) snprintf(err, errlen, "%s", e.msg.c_str());
    *out = nullptr;
    return e.code;
  }
}
void orc_grammar_free(void* g) { delete (Grammar*)g; }
int orc_grammar_num_rules(void* g) { return (int)((Grammar*)g)->rules.size(); }
int orc_grammar_num_nonterminals(void* g) {
  Grammar* gr = (Grammar*)g;
  std::set<int> used;
  for (auto& r : gr->rules) used.insert(r.lhs);
  return (int)used.size();
}
int orc_grammar_num_dotted(void* g) {
  size_t d = 0;
  for (auto& r : ((Grammar*)g)->rules) d += r.rhs.size() + 1;
  return (int)d;
}
size_t orc_grammar_rule_text(void* gp, int rule, char* buf, size_t n) {
  Grammar* g = (Grammar*)gp;
  const Rule& r = g->rules[rule];
  std::string s = g->names[r.lhs] + " ->";
  for (auto& x : r.rhs) s += " " + g->sym_text(x);
  if (buf && n) snprintf(buf, n, "%s", s.c_str());
  return s.size();
}

void* orc_vocab_new(const uint8_t* bytes, const uint64_t* offs, uint32_t V, int32_t eos) {
  auto* v = new Vocab;
  v->tok.resize(V);
  for (uint32_t t = 0; t < V; ++t) v->tok[t].assign((const char*)bytes + offs[t], (size_t)(offs[t + 1] - offs[t]));
  v->eos = eos;
  return v;
}
void orc_vocab_free(void* v) { delete (Vocab*)v; }

void* orc_seq_new(void* g, int pruned) { return new Seq((Grammar*)g, pruned != 0); }
void* orc_seq_clone(void* s) { return new Seq(*(Seq*)s); }
void orc_seq_free(void* s) { delete (Seq*)s; }
int orc_seq_advance(void* s, const uint8_t* bytes, size_t n) { return ((Seq*)s)->advance(bytes, n) ? 1 : 0; }
int orc_seq_accepting(void* s) { return ((Seq*)s)->accepting ? 1 : 0; }
size_t orc_seq_num_sets(void* s) { return ((Seq*)s)->chart.size(); }
size_t orc_seq_set_size(void* s, size_t k) { return ((Seq*)s)->chart[k].items.size(); }
size_t orc_seq_total_items(void* s) { return ((Seq*)s)->total_items(); }
size_t orc_seq_peak_items(void* s) { return ((Seq*)s)->peak_items; }
size_t orc_seq_set_text(void* s, size_t k, char* buf, size_t n) {
  std::string t = ((Seq*)s)->set_text(k);
  if (buf && n) snprintf(buf, n, "%s", t.c_str());
  return t.size();
}
size_t orc_seq_key_text(void* s, char* buf, size_t n) {
  std::string t = ((Seq*)s)->key_text();
  if (buf && n) snprintf(buf, n, "%s", t.c_str());
  return t.size();
}

// Is the one token `bytes` valid after the sequence's prefix?  (non-empty token)
int orc_seq_check_bytes(void* sp, const uint8_t* bytes, size_t n) {
  Seq* s = (Seq*)sp;
  if (n == 0) return 0;
  std::vector<ItemSet> ext;
  return s->extend(bytes, n, ext) ? 1 : 0;
}

// The whole-vocabulary mask: every token checked on its own (Section 4.1: "process all
// tokens in the vocabulary along with already generated tokens").  Bit t&31 of word t>>5.
void orc_seq_mask(void* sp, void* vp, uint32_t* out, int nthreads) {
  Seq* s = (Seq*)sp;
  Vocab* v = (Vocab*)vp;
  size_t V = v->tok.size();
  size_t W = (V + 31) / 32;
  std::vector<unsigned char> valid(V, 0);
#ifdef _OPENMP
  if (nthreads <= 0) nthreads = omp_get_max_threads();
#pragma omp parallel num_threads(nthreads)
#endif
  {
    std::vector<ItemSet> ext;
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 64)
#endif
    for (long t = 0; t < (long)V; ++t) {
      const std::string& b = v->tok[t];
      if ((int)t == v->eos) valid[t] = s->accepting ? 1 : 0;
      else if (b.empty()) valid[t] = 0;
      else valid[t] = s->extend((const unsigned char*)b.data(), b.size(), ext) ? 1 : 0;
    }
  }
  for (size_t w = 0; w < W; ++w) out[w] = 0;
  for (size_t t = 0; t < V; ++t)
    if (valid[t]) out[t >> 5] |= (1u << (t & 31));
}

int orc_max_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Section 3.3: the logit of every token the mask rules out becomes -inf.  dtype 0 = bfloat16, 1 = float32.
// Valid entries are left untouched bit for bit.
void orc_apply_mask(const uint32_t* mask, size_t stride_words, void* logits, int dtype, uint32_t batch, uint32_t V,
                    size_t row_stride_elems) {
  for (uint32_t b = 0; b < batch; ++b)
    for (uint32_t t = 0; t < V; ++t) {
      bool ok = (mask[(size_t)b * stride_words + (t >> 5)] >> (t & 31)) & 1u;
      if (ok) continue;
      if (dtype == 0) ((uint16_t*)logits)[(size_t)b * row_stride_elems + t] = 0xFF80u;
      else ((uint32_t*)logits)[(size_t)b * row_stride_elems + t] = 0xFF800000u;
    }
}

}  // extern "C"
