// JSON Schema (a subset) -> grammar text in this library's EBNF dialect, so that a schema can be
// handed to fmt_compile directly (the paper's JSON-Schema workload, Section 5.1; the paper leaves
// the translation to its front end and fixes none).  Host code only.
//
// What a schema node may hold:
//   "type": "object" | "array" | "string" | "number" | "integer" | "boolean" | "null", or a list of them
//   "properties" (members appear in the order written), "required"; other members are not allowed
//   "items", "minItems" (0 or 1);  "enum", "const";  "anyOf" / "oneOf" (both read as "any of")
//   "$ref": "#/$defs/NAME" or "#/definitions/NAME" (recursion is fine: the target is a CFG)
// A node with none of these accepts any JSON value.  Anything else that would restrict the
// instances (pattern, minimum, maxLength, additionalProperties: true, ...) is refused rather than
// silently ignored, except the annotations title / description / default / examples / $schema / $id.
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <map>
#include <set>
#include <string>
#include <utility>
#include <vector>

#include "../../include/fmt.h"
#include "host_tables.h"

namespace fmt {
namespace {

struct JV {
  enum Kind { Null, Bool, Num, Str, Arr, Obj } kind = Null;
  bool b = false;
  std::string text;  // Num: as written; Str: decoded bytes (UTF-8)
  std::vector<JV> arr;
  std::vector<std::pair<std::string, JV>> obj;  // in the order written
  const JV* get(const char* key) const {
    for (const auto& kv : obj)
      if (kv.first == key) return &kv.second;
    return nullptr;
  }
};

[[noreturn]] void bad(const std::string& msg) { throw CompileError{FMT_ERR_GRAMMAR_SYNTAX, "JSON schema: " + msg}; }

struct Parser {
  const char* p;
  const char* e;
  int depth = 0;
  void ws() {
    while (p < e && (*p == ' ' || *p == '\t' || *p == '\n' || *p == '\r')) ++p;
  }
  void put_utf8(std::string& s, uint32_t c) {
    if (c < 0x80) s += (char)c;
    else if (c < 0x800) s += (char)(0xC0 | (c >> 6)), s += (char)(0x80 | (c & 0x3F));
    else if (c < 0x10000) s += (char)(0xE0 | (c >> 12)), s += (char)(0x80 | ((c >> 6) & 0x3F)), s += (char)(0x80 | (c & 0x3F));
    else s += (char)(0xF0 | (c >> 18)), s += (char)(0x80 | ((c >> 12) & 0x3F)), s += (char)(0x80 | ((c >> 6) & 0x3F)), s += (char)(0x80 | (c & 0x3F));
  }
  uint32_t hex4() {
    if (e - p < 4) bad("truncated \\u escape");
    uint32_t v = 0;
    for (int i = 0; i < 4; ++i) {
      const char c = *p++;
      v <<= 4;
      if (c >= '0' && c <= '9') v |= c - '0';
      else if (c >= 'a' && c <= 'f') v |= c - 'a' + 10;
      else if (c >= 'A' && c <= 'F') v |= c - 'A' + 10;
      else bad("bad \\u escape");
    }
    return v;
  }
  std::string string() {
    if (p >= e || *p != '"') bad("a string was expected");
    ++p;
    std::string s;
    for (;;) {
      if (p >= e) bad("unterminated string");
      const unsigned char c = (unsigned char)*p++;
      if (c == '"') return s;
      if (c < 0x20) bad("control character in a string");
      if (c != '\\') {
        s += (char)c;
        continue;
      }
      if (p >= e) bad("unterminated string");
      const char x = *p++;
      switch (x) {
        case '"': s += '"'; break;
        case '\\': s += '\\'; break;
        case '/': s += '/'; break;
        case 'b': s += '\b'; break;
        case 'f': s += '\f'; break;
        case 'n': s += '\n'; break;
        case 'r': s += '\r'; break;
        case 't': s += '\t'; break;
        case 'u': {
          uint32_t c1 = hex4();
          if (c1 >= 0xD800 && c1 < 0xDC00 && e - p >= 6 && p[0] == '\\' && p[1] == 'u') {
            p += 2;
            const uint32_t c2 = hex4();
            if (c2 < 0xDC00 || c2 > 0xDFFF) bad("unpaired surrogate");
            c1 = 0x10000 + ((c1 - 0xD800) << 10) + (c2 - 0xDC00);
          } else if (c1 >= 0xD800 && c1 <= 0xDFFF) {
            bad("unpaired surrogate");
          }
          put_utf8(s, c1);
          break;
        }
        default: bad("bad escape in a string");
      }
    }
  }
  JV value() {
    if (++depth > 200) bad("nested too deeply");
    ws();
    if (p >= e) bad("unexpected end");
    JV v;
    const char c = *p;
    if (c == '{') {
      ++p;
      v.kind = JV::Obj;
      ws();
      if (p < e && *p == '}') {
        ++p;
      } else {
        for (;;) {
          ws();
          std::string k = string();
          ws();
          if (p >= e || *p != ':') bad("':' expected");
          ++p;
          JV x = value();
          v.obj.emplace_back(std::move(k), std::move(x));
          ws();
          if (p < e && *p == ',') {
            ++p;
            continue;
          }
          if (p < e && *p == '}') {
            ++p;
            break;
          }
          bad("',' or '}' expected");
        }
      }
    } else if (c == '[') {
      ++p;
      v.kind = JV::Arr;
      ws();
      if (p < e && *p == ']') {
        ++p;
      } else {
        for (;;) {
          v.arr.push_back(value());
          ws();
          if (p < e && *p == ',') {
            ++p;
            continue;
          }
          if (p < e && *p == ']') {
            ++p;
            break;
          }
          bad("',' or ']' expected");
        }
      }
    } else if (c == '"') {
      v.kind = JV::Str;
      v.text = string();
    } else if (e - p >= 4 && !memcmp(p, "true", 4)) {
      v.kind = JV::Bool, v.b = true, p += 4;
    } else if (e - p >= 5 && !memcmp(p, "false", 5)) {
      v.kind = JV::Bool, v.b = false, p += 5;
    } else if (e - p >= 4 && !memcmp(p, "null", 4)) {
      v.kind = JV::Null, p += 4;
    } else {
      const char* s = p;
      if (p < e && *p == '-') ++p;
      if (p >= e || *p < '0' || *p > '9') bad("a value was expected");
      if (*p == '0') ++p;
      else
        while (p < e && *p >= '0' && *p <= '9') ++p;
      if (p < e && *p == '.') {
        ++p;
        if (p >= e || *p < '0' || *p > '9') bad("bad number");
        while (p < e && *p >= '0' && *p <= '9') ++p;
      }
      if (p < e && (*p == 'e' || *p == 'E')) {
        ++p;
        if (p < e && (*p == '+' || *p == '-')) ++p;
        if (p >= e || *p < '0' || *p > '9') bad("bad number");
        while (p < e && *p >= '0' && *p <= '9') ++p;
      }
      v.kind = JV::Num;
      v.text.assign(s, p);
    }
    --depth;
    return v;
  }
};

// the bytes `s` as a literal of the grammar dialect
std::string lit(const std::string& s) {
  std::string out = "\"";
  char buf[8];
  for (unsigned char c : s) {
    if (c == '"') out += "\\\"";
    else if (c == '\\') out += "\\\\";
    else if (c >= 0x20 && c < 0x7F) out += (char)c;
    else snprintf(buf, sizeof buf, "\\x%02x", c), out += buf;
  }
  return out + "\"";
}

// the JSON text of a string value, as this library spells it: '"', the bytes with '"', '\' and
// control characters escaped, '"'
std::string json_string_text(const std::string& s) {
  std::string out = "\"";
  char buf[8];
  for (unsigned char c : s) {
    if (c == '"') out += "\\\"";
    else if (c == '\\') out += "\\\\";
    else if (c < 0x20) snprintf(buf, sizeof buf, "\\u%04x", c), out += buf;
    else out += (char)c;
  }
  return out + "\"";
}

// the JSON text of a constant (enum member, const), compact
std::string json_text(const JV& v) {
  switch (v.kind) {
    case JV::Null: return "null";
    case JV::Bool: return v.b ? "true" : "false";
    case JV::Num: return v.text;
    case JV::Str: return json_string_text(v.text);
    case JV::Arr: {
      std::string s = "[";
      for (size_t i = 0; i < v.arr.size(); ++i) s += (i ? "," : "") + json_text(v.arr[i]);
      return s + "]";
    }
    case JV::Obj: {
      std::string s = "{";
      for (size_t i = 0; i < v.obj.size(); ++i) s += (i ? "," : "") + json_string_text(v.obj[i].first) + ":" + json_text(v.obj[i].second);
      return s + "}";
    }
  }
  return "null";
}

struct Emitter {
  const JV& root;
  std::vector<std::string> rules;
  std::map<std::string, std::string> defs;  // "#/$defs/x" -> rule name
  int counter = 0;
  bool need_value = false;
  explicit Emitter(const JV& r) : root(r) {}

  std::string fresh(const char* stem) { return std::string(stem) + std::to_string(counter++); }

  void check_keys(const JV& n) {
    static const std::set<std::string> known = {"type", "properties", "required", "items", "minItems", "enum", "const",
                                                "anyOf", "oneOf", "$ref", "$defs", "definitions", "title", "description",
                                                "default", "examples", "$schema", "$id", "additionalProperties"};
    for (const auto& kv : n.obj)
      if (!known.count(kv.first)) bad("keyword \"" + kv.first + "\" is not supported");
    if (const JV* ap = n.get("additionalProperties"))
      if (!(ap->kind == JV::Bool && !ap->b)) bad("additionalProperties must be false or absent (other members are never allowed)");
  }

  std::string ref(const std::string& target) {
    auto it = defs.find(target);
    if (it != defs.end()) return it->second;
    const JV* node = nullptr;
    for (const char* sect : {"$defs", "definitions"}) {
      const std::string prefix = std::string("#/") + sect + "/";
      if (target.compare(0, prefix.size(), prefix) == 0)
        if (const JV* d = root.get(sect))
          if (d->kind == JV::Obj) node = d->get(target.c_str() + prefix.size());
    }
    if (!node) bad("cannot resolve $ref \"" + target + "\"");
    const std::string name = fresh("def");
    defs[target] = name;  // before the body: the definition may refer to itself
    const std::string body = schema(*node);
    rules.push_back(name + " ::= " + body);
    return name;
  }

  std::string of_type(const JV& n, const std::string& t) {
    if (t == "string") return "string";
    if (t == "number") return "number";
    if (t == "integer") return "integer";
    if (t == "boolean") return "boolean";
    if (t == "null") return "\"null\"";
    if (t == "array") {
      std::string item = "value";
      if (const JV* it = n.get("items")) {
        if (it->kind != JV::Obj) bad("\"items\" must be a schema");
        item = schema(*it);
      } else {
        need_value = true;
      }
      int min_items = 0;
      if (const JV* mi = n.get("minItems")) {
        if (mi->kind != JV::Num || (mi->text != "0" && mi->text != "1")) bad("minItems must be 0 or 1");
        min_items = mi->text == "1";
      }
      const std::string name = fresh("arr");
      const std::string some = "\"[\" ws " + item + " ws ( \",\" ws " + item + " ws )* \"]\"";
      rules.push_back(name + " ::= " + (min_items ? some : "\"[\" ws \"]\" | " + some));
      return name;
    }
    if (t == "object") {
      const JV* props = n.get("properties");
      if (props && props->kind != JV::Obj) bad("\"properties\" must be an object");
      std::set<std::string> required;
      if (const JV* rq = n.get("required")) {
        if (rq->kind != JV::Arr) bad("\"required\" must be a list");
        for (const JV& r : rq->arr) {
          if (r.kind != JV::Str) bad("\"required\" must list strings");
          required.insert(r.text);
        }
      }
      const size_t nf = props ? props->obj.size() : 0;
      for (const std::string& r : required) {
        bool found = false;
        for (size_t i = 0; i < nf; ++i) found |= props->obj[i].first == r;
        if (!found) bad("required member \"" + r + "\" is not among the properties");
      }
      // members in the order written.  first_i: members from the i-th on, none written yet;
      // rest_i: the same after at least one member (a comma comes first)
      const std::string k = std::to_string(counter++);
      const std::string name = "obj" + k;
      rules.push_back(name + " ::= \"{\" ws first" + k + "_0 ws \"}\"");
      for (size_t i = 0; i < nf; ++i) {
        const std::string fld = "fld" + k + "_" + std::to_string(i);
        const std::string ty = schema(props->obj[i].second);
        rules.push_back(fld + " ::= " + lit(json_string_text(props->obj[i].first)) + " ws \":\" ws " + ty);
        const std::string next = k + "_" + std::to_string(i + 1);
        const bool req = required.count(props->obj[i].first) != 0;
        rules.push_back("first" + k + "_" + std::to_string(i) + " ::= " + fld + " rest" + next + (req ? "" : " | first" + next));
        if (i > 0) rules.push_back("rest" + k + "_" + std::to_string(i) + " ::= ws \",\" ws " + fld + " rest" + next + (req ? "" : " | rest" + next));
      }
      rules.push_back("first" + k + "_" + std::to_string(nf) + " ::= \"\"");
      rules.push_back("rest" + k + "_" + std::to_string(nf) + " ::= \"\"");
      return name;
    }
    bad("unknown type \"" + t + "\"");
  }

  // an expression of the dialect for the instances of schema node n
  std::string schema(const JV& n) {
    if (n.kind == JV::Bool) {
      if (!n.b) bad("the schema \"false\" has no instances");
      need_value = true;
      return "value";
    }
    if (n.kind != JV::Obj) bad("a schema must be an object");
    check_keys(n);
    if (const JV* r = n.get("$ref")) {
      if (r->kind != JV::Str) bad("\"$ref\" must be a string");
      return ref(r->text);
    }
    if (const JV* c = n.get("const")) return lit(json_text(*c));
    if (const JV* en = n.get("enum")) {
      if (en->kind != JV::Arr || en->arr.empty()) bad("\"enum\" must be a non-empty list");
      const std::string name = fresh("enum");
      std::string body;
      for (size_t i = 0; i < en->arr.size(); ++i) body += (i ? " | " : "") + lit(json_text(en->arr[i]));
      rules.push_back(name + " ::= " + body);
      return name;
    }
    for (const char* key : {"anyOf", "oneOf"}) {
      if (const JV* alts = n.get(key)) {
        if (alts->kind != JV::Arr || alts->arr.empty()) bad(std::string("\"") + key + "\" must be a non-empty list");
        const std::string name = fresh("any");
        std::string body;
        for (size_t i = 0; i < alts->arr.size(); ++i) body += (i ? " | " : "") + schema(alts->arr[i]);
        rules.push_back(name + " ::= " + body);
        return name;
      }
    }
    const JV* t = n.get("type");
    if (!t) {
      if (n.get("properties")) return of_type(n, "object");
      if (n.get("items")) return of_type(n, "array");
      need_value = true;
      return "value";
    }
    if (t->kind == JV::Str) return of_type(n, t->text);
    if (t->kind != JV::Arr || t->arr.empty()) bad("\"type\" must be a string or a non-empty list of strings");
    const std::string name = fresh("any");
    std::string body;
    for (size_t i = 0; i < t->arr.size(); ++i) {
      if (t->arr[i].kind != JV::Str) bad("\"type\" must list strings");
      body += (i ? " | " : "") + of_type(n, t->arr[i].text);
    }
    rules.push_back(name + " ::= " + body);
    return name;
  }
};

const char* const kCommonRules = R"(boolean ::= "true" | "false"
ws      ::= [ \t\n\r]*
string  ::= "\"" chars "\""
chars   ::= "" | chars char
char    ::= [\x20-\x21\x23-\x5b\x5d-\x7f] | "\\" escape | utf8
escape  ::= ["\\/bfnrt] | "u" hex hex hex hex
hex     ::= [0-9a-fA-F]
utf8    ::= [\xc2-\xdf] cont
          | "\xe0" [\xa0-\xbf] cont | [\xe1-\xec\xee-\xef] cont cont | "\xed" [\x80-\x9f] cont
          | "\xf0" [\x90-\xbf] cont cont | [\xf1-\xf3] cont cont cont | "\xf4" [\x80-\x8f] cont cont
cont    ::= [\x80-\xbf]
number  ::= integer frac? exp?
integer ::= "-"? ( "0" | [1-9] [0-9]* )
frac    ::= "." [0-9]+
exp     ::= [eE] [+\-]? [0-9]+
)";

const char* const kValueRules = R"(value    ::= object | array | string | number | "true" | "false" | "null"
object   ::= "{" ws "}" | "{" members "}"
members  ::= pair | members "," pair
pair     ::= ws string ws ":" ws value ws
array    ::= "[" ws "]" | "[" elements "]"
elements ::= element | elements "," element
element  ::= ws value ws
)";

}  // namespace

std::string json_schema_to_ebnf(const char* text, size_t len) {
  Parser ps{text, text + len};
  const JV root = ps.value();
  ps.ws();
  if (ps.p != ps.e) bad("text after the schema");
  Emitter em(root);
  const std::string top = em.schema(root);
  std::string out = "# generated from a JSON schema; start rule: root\nroot ::= ws " + top + " ws\n";
  for (const std::string& r : em.rules) out += r + "\n";
  out += kCommonRules;
  if (em.need_value) out += kValueRules;
  return out;
}

}  // namespace fmt
