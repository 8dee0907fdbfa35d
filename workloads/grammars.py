"""The five synthetic grammars (EBNF text) and a hand-written document generator
for each, so that every generated document is a sentence of its grammar.

Dialect of the grammar text (both the CPU oracle and the CUDA library parse it
with parsers of their own):

    name ::= alternative ( "|" alternative )*
    alternative = sequence of: "literal"  [byte class]  name  ( group )  with postfix * + ?
    "" is the empty string; # starts a comment; a rule ends where the next `name ::=` starts
    escapes in literals and classes: \\xHH \\n \\r \\t \\\\ \\" \\] \\- \\^

This module only produces text and bytes; it contains no parsing or masking logic.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Tuple

from .rng import SplitMix64

# --------------------------------------------------------------------------- config 1

ARITH_EBNF = r"""
# arithmetic expressions, left recursive
expr   ::= expr [+\-] term | term
term   ::= term [*/] factor | factor
factor ::= "(" expr ")" | number
number ::= [0-9]+
"""


def gen_arith(rng: SplitMix64, depth: int = 0, max_depth: int = 5) -> bytes:
    def number() -> bytes:
        n = 1 + rng.geometric(1.5)
        return bytes(0x30 + rng.below(10) for _ in range(min(n, 6)))

    def factor(d: int) -> bytes:
        if d < max_depth and rng.chance(0.3):
            return b"(" + expr(d + 1) + b")"
        return number()

    def term(d: int) -> bytes:
        out = factor(d)
        while rng.chance(0.35):
            out += rng.pick([b"*", b"/"]) + factor(d)
        return out

    def expr(d: int) -> bytes:
        out = term(d)
        while rng.chance(0.45):
            out += rng.pick([b"+", b"-"]) + term(d)
        return out

    return expr(depth)


def gen_arith_doc(rng: SplitMix64) -> bytes:
    # long enough for a 64-byte prefix plus 32 tokens
    parts = [gen_arith(rng)]
    while sum(len(p) for p in parts) < 260:
        parts.append(rng.pick([b"+", b"-", b"*", b"/"]))
        parts.append(gen_arith(rng))
    return b"".join(parts)


# --------------------------------------------------------------------------- config 2

_JSON_STRING_RULES = r"""
string ::= "\"" chars "\""
chars  ::= "" | chars char
char   ::= [\x20-\x21\x23-\x5b\x5d-\x7f] | "\\" escape | utf8
escape ::= ["\\/bfnrt] | "u" hex hex hex hex
hex    ::= [0-9a-fA-F]
utf8   ::= [\xc2-\xdf] cont
         | "\xe0" [\xa0-\xbf] cont | [\xe1-\xec\xee-\xef] cont cont | "\xed" [\x80-\x9f] cont
         | "\xf0" [\x90-\xbf] cont cont | [\xf1-\xf3] cont cont cont | "\xf4" [\x80-\x8f] cont cont
cont   ::= [\x80-\xbf]
"""

_JSON_NUMBER_RULES = r"""
number  ::= integer frac? exp?
integer ::= "-"? ( "0" | [1-9] [0-9]* )
frac    ::= "." [0-9]+
exp     ::= [eE] [+\-]? [0-9]+
"""

JSON_EBNF = (
    r"""
# JSON (RFC 8259), byte level, UTF-8 spelled out
json     ::= ws value ws
value    ::= object | array | string | number | "true" | "false" | "null"
object   ::= "{" ws "}" | "{" members "}"
members  ::= pair | members "," pair
pair     ::= ws string ws ":" ws value ws
array    ::= "[" ws "]" | "[" elements "]"
elements ::= element | elements "," element
element  ::= ws value ws
ws       ::= [ \t\n\r]*
"""
    + _JSON_STRING_RULES
    + _JSON_NUMBER_RULES
)

_WORD_CHARS = b"abcdefghijklmnopqrstuvwxyzABCDEFGHIJKLMNOPQRSTUVWXYZ0123456789"
_PUNCT = b" _-.,:;!?/()[]{}<>@#$%&*+='|~^`"


def _utf8_char(rng: SplitMix64) -> bytes:
    r = rng.below(10)
    if r < 6:
        cp = rng.between(0xA0, 0x7FF)
    elif r < 9:
        cp = rng.between(0x800, 0xFFFF)
        if 0xD800 <= cp <= 0xDFFF:
            cp = 0x4E2D
    else:
        cp = rng.between(0x10000, 0x10FFFF)
    return chr(cp).encode("utf-8")


def gen_json_string_body(rng: SplitMix64, mean_len: float = 6.0) -> bytes:
    n = rng.geometric(mean_len)
    out = bytearray()
    for _ in range(min(n, 40)):
        r = rng.below(100)
        if r < 80:
            out.append(rng.pick(_WORD_CHARS))
        elif r < 90:
            out.append(rng.pick(_PUNCT))
        elif r < 94:
            out += _utf8_char(rng)
        elif r < 98:
            out += b"\\" + bytes([rng.pick(b'"\\/bfnrt')])
        else:
            out += b"\\u" + bytes(rng.pick(b"0123456789abcdefABCDEF") for _ in range(4))
    return bytes(out)


def gen_json_number(rng: SplitMix64, integer_only: bool = False) -> bytes:
    out = bytearray()
    if rng.chance(0.2):
        out += b"-"
    if rng.chance(0.15):
        out += b"0"
    else:
        out.append(0x31 + rng.below(9))
        for _ in range(min(rng.geometric(1.5), 8)):
            out.append(0x30 + rng.below(10))
    if not integer_only:
        if rng.chance(0.3):
            out += b"."
            for _ in range(1 + min(rng.geometric(1.0), 5)):
                out.append(0x30 + rng.below(10))
        if rng.chance(0.1):
            out += rng.pick([b"e", b"E"]) + rng.pick([b"", b"+", b"-"])
            for _ in range(1 + rng.below(2)):
                out.append(0x30 + rng.below(10))
    return bytes(out)


def _ws(rng: SplitMix64, p: float = 0.3) -> bytes:
    if not rng.chance(p):
        return b""
    return rng.pick([b" ", b" ", b" ", b"\n", b"\n  ", b"\t", b"\r\n"])


def gen_json_value(rng: SplitMix64, depth: int, max_depth: int, extra=None) -> bytes:
    """A random JSON value.  `extra(rng, depth)` may return bytes for an extra
    alternative of `value` (config 5), or None."""
    if extra is not None:
        e = extra(rng, depth)
        if e is not None:
            return e
    if depth >= max_depth:
        r = 2 + rng.below(5)
    else:
        r = rng.below(10)
        r = 0 if r < 3 else 1 if r < 5 else 2 + (r - 5)
    if r == 0:
        n = rng.below(5)
        if n == 0:
            return b"{" + _ws(rng) + b"}"
        pairs = []
        for _ in range(n):
            pairs.append(
                _ws(rng) + b'"' + gen_json_string_body(rng, 4.0) + b'"' + _ws(rng, 0.1) + b":" + _ws(rng, 0.5)
                + gen_json_value(rng, depth + 1, max_depth, extra) + _ws(rng, 0.1)
            )
        return b"{" + b",".join(pairs) + b"}"
    if r == 1:
        n = rng.below(5)
        if n == 0:
            return b"[" + _ws(rng) + b"]"
        els = [_ws(rng) + gen_json_value(rng, depth + 1, max_depth, extra) + _ws(rng, 0.1) for _ in range(n)]
        return b"[" + b",".join(els) + b"]"
    if r == 2 or r == 3:
        return b'"' + gen_json_string_body(rng) + b'"'
    if r == 4:
        return gen_json_number(rng)
    return rng.pick([b"true", b"false", b"null"])


def gen_json_doc(rng: SplitMix64, max_depth: int = 6, min_len: int = 900) -> bytes:
    """A document: an object whose members are random values, at least min_len bytes."""
    pairs = []
    total = 0
    while total < min_len:
        p = (
            _ws(rng) + b'"' + gen_json_string_body(rng, 4.0) + b'"' + b":" + _ws(rng, 0.5)
            + gen_json_value(rng, 1, max_depth) + _ws(rng, 0.1)
        )
        pairs.append(p)
        total += len(p) + 1
    return _ws(rng, 0.1) + b"{" + b",".join(pairs) + b"}" + _ws(rng, 0.1)


# --------------------------------------------------------------------------- config 3


def _lit(s: bytes) -> str:
    """EBNF literal for the bytes s."""
    out = ['"']
    for c in s:
        if c == 0x22:
            out.append('\\"')
        elif c == 0x5C:
            out.append("\\\\")
        elif 0x20 <= c < 0x7F:
            out.append(chr(c))
        else:
            out.append("\\x%02x" % c)
    out.append('"')
    return "".join(out)


def _word(rng: SplitMix64, lo: int = 3, hi: int = 10) -> bytes:
    cons = b"bcdfghjklmnprstvwz"
    vow = b"aeiou"
    n = rng.between(lo, hi)
    out = bytearray()
    for i in range(n):
        out.append(rng.pick(cons if i % 2 == 0 else vow))
    return bytes(out)


@dataclass
class SchemaField:
    name: bytes
    required: bool
    kind: str  # string number integer boolean enum object array
    enum: List[bytes] = field(default_factory=list)
    fields: List["SchemaField"] = field(default_factory=list)


def gen_schema(rng: SplitMix64, n_fields: int = 12, depth: int = 1, max_depth: int = 3) -> List[SchemaField]:
    out: List[SchemaField] = []
    used = set()
    for i in range(n_fields):
        while True:
            name = _word(rng)
            if rng.chance(0.3):
                name += rng.pick([b"_", b""]) + _word(rng, 2, 6).capitalize()
            if name not in used:
                used.add(name)
                break
        kinds = ["string", "number", "integer", "boolean", "enum"]
        if depth < max_depth:
            kinds += ["object", "array", "enum", "string"]
        kind = rng.pick(kinds)
        if depth == 1 and i == 3:
            kind = "object"
        if depth == 1 and i == 7:
            kind = "array"
        f = SchemaField(name=name, required=(i == 0) or rng.chance(0.6), kind=kind)
        if kind == "enum":
            vals = set()
            want = rng.between(3, 10)
            while len(vals) < want:
                vals.add(_word(rng, 3, 9))
            f.enum = sorted(vals)
        elif kind in ("object", "array"):
            f.fields = gen_schema(rng, rng.between(2, 4), depth + 1, max_depth)
        out.append(f)
    return out


def schema_to_ebnf(schema: List[SchemaField]) -> str:
    lines: List[str] = ["# generated from a seeded random schema", "root ::= ws obj0 ws"]
    counter = [0]

    def emit_object(fields: List[SchemaField]) -> str:
        k = counter[0]
        counter[0] += 1
        name = "obj%d" % k
        lines.append('%s ::= "{" ws fld%d_0 tail%d_1 ws "}"' % (name, k, k))
        for i, f in enumerate(fields):
            ty = type_ref(f)
            lines.append('fld%d_%d ::= %s ws ":" ws %s' % (k, i, _lit(b'"' + f.name + b'"'), ty))
            if i >= 1:
                body = 'ws "," ws fld%d_%d tail%d_%d' % (k, i, k, i + 1)
                if f.required:
                    lines.append("tail%d_%d ::= %s" % (k, i, body))
                else:
                    lines.append("tail%d_%d ::= %s | tail%d_%d" % (k, i, body, k, i + 1))
        lines.append('tail%d_%d ::= ""' % (k, len(fields)))
        return name

    def type_ref(f: SchemaField) -> str:
        if f.kind in ("string", "number", "integer", "boolean"):
            return f.kind
        if f.kind == "enum":
            k = counter[0]
            counter[0] += 1
            lines.append("enum%d ::= %s" % (k, " | ".join(_lit(b'"' + v + b'"') for v in f.enum)))
            return "enum%d" % k
        sub = emit_object(f.fields)
        if f.kind == "object":
            return sub
        k = counter[0]
        counter[0] += 1
        lines.append('arr%d ::= "[" ws "]" | "[" ws %s ws ( "," ws %s ws )* "]"' % (k, sub, sub))
        return "arr%d" % k

    emit_object(schema)
    lines.append('boolean ::= "true" | "false"')
    lines.append("ws ::= [ \\t\\n\\r]*")
    return "\n".join(lines) + "\n" + _JSON_STRING_RULES + _JSON_NUMBER_RULES


def gen_schema_instance(rng: SplitMix64, schema: List[SchemaField], indent: int = 0) -> bytes:
    def ws(p=0.25):
        return _ws(rng, p)

    def value(f: SchemaField) -> bytes:
        if f.kind == "string":
            return b'"' + gen_json_string_body(rng, 8.0) + b'"'
        if f.kind == "number":
            return gen_json_number(rng)
        if f.kind == "integer":
            return gen_json_number(rng, integer_only=True)
        if f.kind == "boolean":
            return rng.pick([b"true", b"false"])
        if f.kind == "enum":
            return b'"' + rng.pick(f.enum) + b'"'
        if f.kind == "object":
            return obj(f.fields)
        n = rng.below(4)
        if n == 0:
            return b"[" + ws() + b"]"
        return b"[" + b",".join(ws() + obj(f.fields) + ws(0.1) for _ in range(n)) + b"]"

    def obj(fields: List[SchemaField]) -> bytes:
        parts = []
        for i, f in enumerate(fields):
            if i > 0 and not f.required and not rng.chance(0.6):
                continue
            parts.append(b'"' + f.name + b'"' + ws(0.05) + b":" + ws(0.5) + value(f))
        body = parts[0]
        for p in parts[1:]:
            body += ws(0.05) + b"," + ws(0.5) + p
        return b"{" + ws() + body + ws() + b"}"

    return ws(0.1) + obj(schema) + ws(0.1)


# --------------------------------------------------------------------------- config 4


def gen_sql_names(rng: SplitMix64) -> Tuple[List[bytes], List[bytes]]:
    tabs, cols = set(), set()
    while len(tabs) < 60:
        tabs.add(b"t_" + _word(rng, 3, 8))
    while len(cols) < 140:
        c = _word(rng, 3, 8)
        if rng.chance(0.3):
            c += b"_" + rng.pick([b"id", b"at", b"name", b"count", b"ts"])
        cols.add(b"c_" + c if rng.chance(0.5) else c)
    return sorted(tabs), sorted(cols)


_SQL_KEYWORDS = {
    b"select", b"from", b"where", b"join", b"left", b"right", b"inner", b"group", b"order", b"by", b"having",
    b"limit", b"and", b"or", b"not", b"in", b"is", b"null", b"like", b"between", b"as", b"on", b"asc", b"desc",
    b"count", b"sum", b"avg", b"min", b"max", b"distinct",
}


def sql_ebnf(tabs: List[bytes], cols: List[bytes]) -> str:
    head = r"""
# SQL-like semantic-parsing DSL
query      ::= select_stmt ";"?
select_stmt ::= "SELECT " distinct? select_list " FROM " table_ref join* where? group? order? limit?
distinct   ::= "DISTINCT "
select_list ::= "*" | select_item ( "," sp select_item )*
select_item ::= expr alias?
alias      ::= " AS " colname
table_ref  ::= tabname tab_alias?
tab_alias  ::= " " tabalias
join       ::= join_kind "JOIN " table_ref " ON " cond
join_kind  ::= " " | " LEFT " | " INNER " | " RIGHT "
where      ::= " WHERE " cond
group      ::= " GROUP BY " colref ( "," sp colref )* having?
having     ::= " HAVING " cond
order      ::= " ORDER BY " order_item ( "," sp order_item )*
order_item ::= colref ( " ASC" | " DESC" )?
limit      ::= " LIMIT " uint
cond       ::= cond " OR " cond_and | cond_and
cond_and   ::= cond_and " AND " cond_not | cond_not
cond_not   ::= "NOT " cond_not | pred
pred       ::= expr cmp expr
             | expr " IS NULL" | expr " IS NOT NULL"
             | expr " IN (" expr_list ")"
             | expr " BETWEEN " expr " AND " expr
             | expr " LIKE " sqlstring
             | "(" cond ")"
cmp        ::= " = " | " <> " | " < " | " > " | " <= " | " >= "
expr_list  ::= expr ( "," sp expr )*
expr       ::= expr " + " term | expr " - " term | term
term       ::= term " * " factor | term " / " factor | factor
factor     ::= colref | number | sqlstring | func "(" func_arg ")" | "(" expr ")" | "-" factor
func       ::= "COUNT" | "SUM" | "AVG" | "MIN" | "MAX"
func_arg   ::= "*" | expr | "DISTINCT " expr
colref     ::= colname | tabname "." colname | tabalias "." colname
tabalias   ::= [a-z] [0-9]
sqlstring  ::= "'" sqlchar* "'"
sqlchar    ::= [\x20-\x26\x28-\x7e] | "''"
number     ::= uint ( "." [0-9]+ )?
uint       ::= [0-9]+
sp         ::= " "?
"""
    t = "tabname ::= " + " | ".join(_lit(x) for x in tabs)
    c = "colname ::= " + " | ".join(_lit(x) for x in cols)
    return head + t + "\n" + c + "\n"


def gen_sql_doc(rng: SplitMix64, tabs: List[bytes], cols: List[bytes], max_len: int = 400) -> bytes:
    aliases: List[bytes] = []

    def sp() -> bytes:
        return b" " if rng.chance(0.7) else b""

    def colref() -> bytes:
        r = rng.below(10)
        if r < 5 or (r >= 8 and not aliases):
            return rng.pick(cols)
        if r < 8:
            return rng.pick(tabs) + b"." + rng.pick(cols)
        return rng.pick(aliases) + b"." + rng.pick(cols)

    def number() -> bytes:
        out = bytes(0x30 + rng.below(10) for _ in range(1 + min(rng.geometric(1.0), 5)))
        if rng.chance(0.2):
            out += b"." + bytes(0x30 + rng.below(10) for _ in range(1 + rng.below(3)))
        return out

    def sqlstring() -> bytes:
        n = min(rng.geometric(5.0), 16)
        out = bytearray(b"'")
        for _ in range(n):
            if rng.chance(0.03):
                out += b"''"
            else:
                c = rng.between(0x20, 0x7E)
                out.append(0x41 if c == 0x27 else c)
        return bytes(out) + b"'"

    def factor(d: int) -> bytes:
        r = rng.below(20)
        if r < 9:
            return colref()
        if r < 13:
            return number()
        if r < 15:
            return sqlstring()
        if r < 17:
            f = rng.pick([b"COUNT", b"SUM", b"AVG", b"MIN", b"MAX"])
            a = b"*" if rng.chance(0.3) else (b"DISTINCT " if rng.chance(0.2) else b"") + expr(d + 1)
            return f + b"(" + a + b")"
        if r < 19 and d < 3:
            return b"(" + expr(d + 1) + b")"
        return b"-" + colref()

    def term(d: int) -> bytes:
        out = factor(d)
        while rng.chance(0.15):
            out += rng.pick([b" * ", b" / "]) + factor(d)
        return out

    def expr(d: int = 0) -> bytes:
        out = term(d)
        while rng.chance(0.2):
            out += rng.pick([b" + ", b" - "]) + term(d)
        return out

    def pred(d: int) -> bytes:
        r = rng.below(20)
        if r < 10:
            return expr(d) + rng.pick([b" = ", b" <> ", b" < ", b" > ", b" <= ", b" >= "]) + expr(d)
        if r < 12:
            return expr(d) + rng.pick([b" IS NULL", b" IS NOT NULL"])
        if r < 14:
            return expr(d) + b" IN (" + (b"," + sp()).join(expr(d) for _ in range(rng.between(1, 4))) + b")"
        if r < 16:
            return expr(d) + b" BETWEEN " + expr(d) + b" AND " + expr(d)
        if r < 18:
            return expr(d) + b" LIKE " + sqlstring()
        if d < 2:
            return b"(" + cond(d + 1) + b")"
        return expr(d) + b" = " + expr(d)

    def cond_not(d: int) -> bytes:
        return (b"NOT " if rng.chance(0.1) else b"") + pred(d)

    def cond_and(d: int) -> bytes:
        out = cond_not(d)
        while rng.chance(0.3):
            out += b" AND " + cond_not(d)
        return out

    def cond(d: int = 0) -> bytes:
        out = cond_and(d)
        while rng.chance(0.2):
            out += b" OR " + cond_and(d)
        return out

    def table_ref() -> bytes:
        out = rng.pick(tabs)
        if rng.chance(0.5):
            a = bytes([0x61 + rng.below(26), 0x30 + rng.below(10)])
            aliases.append(a)
            out += b" " + a
        return out

    for _ in range(20):
        aliases.clear()
        from_part = b" FROM " + table_ref()
        for _j in range(rng.below(3)):
            from_part += rng.pick([b" ", b" LEFT ", b" INNER ", b" RIGHT "]) + b"JOIN " + table_ref() + b" ON " + cond(1)
        out = b"SELECT " + (b"DISTINCT " if rng.chance(0.15) else b"")
        if rng.chance(0.15):
            out += b"*"
        else:
            items = []
            for _j in range(rng.between(1, 4)):
                it = expr()
                if rng.chance(0.25):
                    it += b" AS " + rng.pick(cols)
                items.append(it)
            out += (b"," + sp()).join(items)
        out += from_part
        if rng.chance(0.7):
            out += b" WHERE " + cond()
        if rng.chance(0.3):
            out += b" GROUP BY " + (b"," + sp()).join(colref() for _j in range(rng.between(1, 3)))
            if rng.chance(0.4):
                out += b" HAVING " + cond(1)
        if rng.chance(0.4):
            out += b" ORDER BY " + (b"," + sp()).join(
                colref() + rng.pick([b"", b" ASC", b" DESC"]) for _j in range(rng.between(1, 3))
            )
        if rng.chance(0.3):
            out += b" LIMIT " + bytes(0x31 + rng.below(9) for _j in range(rng.between(1, 3)))
        if rng.chance(0.5):
            out += b";"
        if len(out) <= max_len:
            return out
    return b"SELECT * FROM " + tabs[0]


# --------------------------------------------------------------------------- config 5

N_CHAIN = 12  # N0..N11


def stress_ebnf() -> str:
    chain = []
    for i in range(N_CHAIN - 2):
        chain.append('N%d ::= N%d N%d | ""' % (i, i + 1, i + 2))
    chain.append('N%d ::= "_" | ""' % (N_CHAIN - 2))
    chain.append('N%d ::= "~" | ""' % (N_CHAIN - 1))
    extra = r"""
# ambiguity and nullable stress, embedded in JSON as the value alternative "<" amb ">"
amb  ::= W E W
E    ::= E E | E O3 "+" O3 E | "(" W E W ")" | "a" | "b"
W    ::= N0 | O4
O1   ::= "!"?
O2   ::= O1 O1
O3   ::= O2 | "" | O1 O2
O4   ::= O3 O3 | O1
O5   ::= "," ws | ""
O6   ::= O5
pad  ::= O6 O6
""" + "\n".join(chain) + "\n"
    base = JSON_EBNF.replace('| "true" | "false" | "null"', '| "true" | "false" | "null" | "<" amb ">"')
    assert base != JSON_EBNF
    return base + extra


def gen_amb_segment(rng: SplitMix64, max_len: int = 96) -> bytes:
    """A sentence of `amb` of at most max_len bytes."""

    def w() -> bytes:
        if rng.chance(0.75):
            return b""
        if rng.chance(0.5):
            return bytes(rng.pick(b"_~") for _ in range(rng.between(1, 4)))  # within N0's reach in any order
        return b"!" * rng.between(1, 3)

    def o3() -> bytes:
        return b"!" * rng.below(3) if rng.chance(0.2) else b""

    def e(budget: int, d: int) -> bytes:
        if budget <= 2 or d > 6:
            return rng.pick([b"a", b"b"])
        r = rng.below(10)
        if r < 4:
            left = e(budget // 2, d + 1)
            return left + e(budget - len(left), d + 1)
        if r < 6:
            left = e(budget // 2 - 2, d + 1)
            return left + o3() + b"+" + o3() + e(budget - len(left) - 6, d + 1)
        if r < 8 and budget > 12:
            return b"(" + w() + e(budget - 10, d + 1) + w() + b")"
        return rng.pick([b"a", b"b"])

    for _ in range(50):
        s = w() + e(max_len - 10, 0) + w()
        if len(s) <= max_len:
            return s
    return b"a"


# N0 derives a string over {_,~} only along its Fibonacci-like tree; not every order/length is
# derivable, so the generator above must stay inside what W really derives.  The set below is
# produced by brute force once and used to filter W runs.
def _n_chain_language(max_len: int = 4):
    lang = [set() for _ in range(N_CHAIN)]
    lang[N_CHAIN - 2] = {b"_", b""}
    lang[N_CHAIN - 1] = {b"~", b""}
    for i in range(N_CHAIN - 3, -1, -1):
        s = {b""}
        for a in lang[i + 1]:
            for b in lang[i + 2]:
                if len(a) + len(b) <= max_len:
                    s.add(a + b)
        lang[i] = s
    return lang[0]


_W_RUNS = None


def w_runs():
    global _W_RUNS
    if _W_RUNS is None:
        _W_RUNS = sorted(x for x in _n_chain_language(4) if x)
    return _W_RUNS


def gen_amb_segment_checked(rng: SplitMix64, max_len: int = 96) -> bytes:
    """gen_amb_segment with every `_~` run replaced by one W really derives."""
    runs = w_runs()
    s = gen_amb_segment(rng, max_len)
    out = bytearray()
    i = 0
    while i < len(s):
        if s[i] in b"_~":
            j = i
            while j < len(s) and s[j] in b"_~":
                j += 1
            run = bytes(s[i:j])
            if run not in runs:
                cands = [r for r in runs if len(r) == len(run)] or runs
                run = rng.pick(cands)
            out += run
            i = j
        else:
            out.append(s[i])
            i += 1
    return bytes(out)


def gen_stress_doc(rng: SplitMix64, min_len: int, max_nest: int = 32) -> Tuple[bytes, List[Tuple[int, int]]]:
    """A JSON document of at least min_len bytes with `<amb>` values; returns the
    document and the [start, end) byte spans of the amb segments."""
    spans: List[Tuple[int, int]] = []
    MARK = b"\x00AMB\x00"
    segs: List[bytes] = []

    def extra(r: SplitMix64, depth: int):
        if r.chance(0.18):
            segs.append(gen_amb_segment_checked(r))
            return MARK
        return None

    def deep(r: SplitMix64, d: int) -> bytes:
        # a spine of nested arrays/objects down to depth d
        if d == 0:
            return gen_json_value(r, max_nest - 2, max_nest, extra)
        if r.chance(0.5):
            return b"[" + deep(r, d - 1) + b"," + gen_json_value(r, max_nest - 1, max_nest, extra) + b"]"
        return b'{"' + gen_json_string_body(r, 3.0).replace(b"\x00", b"") + b'":' + deep(r, d - 1) + b"}"

    pairs = []
    total = 0
    while total < min_len:
        if rng.chance(0.15):
            v = deep(rng, rng.between(8, max_nest - 2))
        else:
            v = gen_json_value(rng, 1, 6, extra)
        p = _ws(rng) + b'"' + gen_json_string_body(rng, 4.0) + b'":' + _ws(rng, 0.5) + v + _ws(rng, 0.1)
        pairs.append(p)
        total += len(p) + 1
    doc = b"{" + b",".join(pairs) + b"}"
    # splice the segments in and record spans
    out = bytearray()
    pos = 0
    k = 0
    while True:
        j = doc.find(MARK, pos)
        if j < 0:
            out += doc[pos:]
            break
        out += doc[pos:j]
        out += b"<"
        spans.append((len(out), len(out) + len(segs[k])))
        out += segs[k] + b">"
        k += 1
        pos = j + len(MARK)
    return bytes(out), spans
