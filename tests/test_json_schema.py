"""The JSON-schema front end (fmt_json_schema_to_ebnf / fmt_compile_json_schema): the grammar text it
writes is read by the CPU oracle's own parser and must accept exactly the instances the schema
allows (checked on hand-written instances, valid and invalid, each also run through Python's json
module), and keywords it cannot honour must be refused, not ignored."""
import json

import numpy as np
import pytest

import oracle
import paper_2506_01151_b200 as fmt

SCHEMA = r'''
{
  "$schema": "https://json-schema.org/draft/2020-12/schema",
  "title": "record",
  "type": "object",
  "properties": {
    "name":  {"type": "string", "description": "any JSON string"},
    "age":   {"type": "integer"},
    "score": {"type": ["number", "null"]},
    "kind":  {"enum": ["cat", "do\"g", 3, null, true]},
    "tags":  {"type": "array", "items": {"type": "string"}, "minItems": 1},
    "pos":   {"$ref": "#/$defs/point"},
    "any":   {},
    "fixed": {"const": {"a": [1, "x"]}}
  },
  "required": ["name", "pos"],
  "additionalProperties": false,
  "$defs": {
    "point": {
      "type": "object",
      "properties": {"x": {"type": "number"}, "next": {"anyOf": [{"type": "null"}, {"$ref": "#/$defs/point"}]}},
      "required": ["x"]
    }
  }
}
'''

VALID = [
    '{"name":"a","pos":{"x":1}}',
    ' { "name" : "\\u00e9\\n" , "age" : -12 , "pos" : { "x" : 1.5e3 , "next" : null } } ',
    '{"name":"","score":null,"kind":"do\\"g","tags":["t","u"],"pos":{"x":0,"next":{"x":-0.5,"next":{"x":2}}}}',
    '{"name":"n","kind":3,"pos":{"x":1},"any":[1,{"k":[true,null]},"s"],"fixed":{"a":[1,"x"]}}',
    '{"name":"n","score":2.25,"kind":null,"pos":{"x":1},"any":{}}',
    '{"name":"café","kind":true,"pos":{"x":7}}',
]
INVALID = [
    '{"pos":{"x":1}}',                               # required member missing
    '{"name":"a"}',                                  # required member missing
    '{"pos":{"x":1},"name":"a"}',                    # members out of order
    '{"name":"a","pos":{"x":1},"extra":1}',          # a member the schema does not list
    '{"name":"a","age":1.5,"pos":{"x":1}}',          # not an integer
    '{"name":"a","score":"3","pos":{"x":1}}',        # neither number nor null
    '{"name":"a","kind":"bird","pos":{"x":1}}',      # not in the enum
    '{"name":"a","tags":[],"pos":{"x":1}}',          # minItems 1
    '{"name":"a","tags":["t",1],"pos":{"x":1}}',     # item of the wrong type
    '{"name":"a","pos":{"next":null}}',              # nested required member missing
    '{"name":"a","pos":{"x":1,"next":3}}',           # neither null nor a point
    '{"name":"a","pos":{"x":1},"fixed":{"a":[1]}}',  # not the constant
    '{"name":"a","pos":{"x":1},}',                   # not JSON
    '{"name":"a" "pos":{"x":1}}',                    # not JSON
    '{"name":"a\x01","pos":{"x":1}}',                # control character in a string
]


def accepts(g, text: str) -> bool:
    s = oracle.Sequence_(g)
    return bool(s.advance(text.encode("utf-8"))) and bool(s.accepting)


def test_grammar_accepts_exactly_the_schema_instances():
    ebnf = fmt.json_schema_to_ebnf(SCHEMA)
    g = oracle.Grammar(ebnf, "root")
    for doc in VALID:
        json.loads(doc)
        assert accepts(g, doc), doc
    for doc in INVALID:
        assert not accepts(g, doc), doc
    # every proper prefix of a valid instance stays viable (the mask never goes empty on the way)
    for doc in VALID[:3]:
        data = doc.encode("utf-8")
        s = oracle.Sequence_(g)
        for i in range(len(data)):
            assert s.advance(data[i:i + 1]), (doc, i)


@pytest.mark.parametrize("schema,instances,others", [
    ('{"type":"array","items":{"type":"boolean"}}', ["[]", "[true]", "[ true , false ]"], ["[1]", "[true,]", "{}"]),
    ('{"type":"string"}', ['"x"', '"\\ud83d\\ude00"', '"\U0001F600"'], ["x", '"\\x"', "1"]),
    ('{"oneOf":[{"type":"integer"},{"const":"none"}]}', ["0", "-17", '"none"'], ["01", "1.0", '"None"']),
    ('{"properties":{"a":{"type":"null"},"b":{"type":"null"}}}', ["{}", '{"a":null}', '{"b":null}', '{"a":null,"b":null}'],
     ['{"b":null,"a":null}', '{"a":null,}', '{,"b":null}']),
    ("true", ['{"k":[1,2,{"z":null}]}', "3", '"s"'], ["{", "[1,]"]),
])
def test_small_schemas(schema, instances, others):
    g = oracle.Grammar(fmt.json_schema_to_ebnf(schema), "root")
    for doc in instances:
        json.loads(doc)
        assert accepts(g, doc), doc
    for doc in others:
        assert not accepts(g, doc), doc


@pytest.mark.parametrize("schema", [
    '{"type":"string","pattern":"^a"}',            # a restriction this front end cannot express
    '{"type":"object","additionalProperties":true}',
    '{"type":"array","minItems":3}',
    '{"type":"integer","minimum":0}',
    '{"$ref":"#/$defs/missing"}',
    '{"type":"object","properties":{"a":{}},"required":["b"]}',
    '{"type":"strnig"}',
    '{"type":"string"',                              # not JSON
    "false",
])
def test_what_cannot_be_honoured_is_refused(schema):
    with pytest.raises(fmt.FmtError) as e:
        fmt.json_schema_to_ebnf(schema)
    assert e.value.code == fmt.ERR_GRAMMAR_SYNTAX


def test_compile_json_schema_host_only():
    vocab = [bytes([b]) for b in range(256)] + [b'{"name":', b'"pos"', b"null", b""]
    g = fmt.Grammar.from_json_schema(SCHEMA, vocab, eos=len(vocab) - 1, host_only=True)
    info = g.info()
    assert info.vocab_size == len(vocab) and info.n_rules > 40 and info.n_nullable >= 1
    with pytest.raises(fmt.FmtError):
        fmt.Grammar.from_json_schema('{"type":"string","maxLength":3}', vocab, eos=len(vocab) - 1, host_only=True)


@pytest.mark.gpu
def test_masks_of_a_schema_grammar_equal_the_oracle():
    import torch

    dev = torch.device("cuda:0")
    vocab = [bytes([b]) for b in range(256)] + [b'{"name":', b'"pos"', b'":', b'", "', b"null", b"true", b'{"x":', b"}}", b'"age": ', b""]
    eos = len(vocab) - 1
    g = fmt.Grammar.from_json_schema(SCHEMA, vocab, eos)
    og, ov = oracle.Grammar(fmt.json_schema_to_ebnf(SCHEMA), "root"), oracle.Vocab(vocab, eos)
    st = fmt.State(g, 2)
    docs = [VALID[1].encode(), VALID[2].encode()]
    seqs = [oracle.Sequence_(og) for _ in docs]
    mask = torch.zeros((2, g.mask_words), dtype=torch.int32, device=dev)
    status = torch.zeros(2, dtype=torch.int32, device=dev)
    for i in range(max(len(d) for d in docs)):
        toks = [d[i] if i < len(d) else -1 for d in docs]
        st.advance(torch.tensor(toks, dtype=torch.int32, device=dev), status)
        assert status.cpu().tolist() == [0, 0]
        for b, d in enumerate(docs):
            if i < len(d):
                assert seqs[b].advance(d[i:i + 1])
        st.fill_mask(mask)
        got = mask.cpu().numpy().view(np.uint32)
        for b in range(2):
            assert np.array_equal(got[b], seqs[b].mask(ov)), (i, b)
    assert bool(st.query()["accepting"][1])
