"""Seeded synthetic structural-tag streams (stand-ins for parser transitions on function calls).

The paper tags every generated token from the constrained decoder's parser transition and
groups prompt tokens by input-derived labels. Neither a grammar engine nor the benchmark's
items exist here, so this module invents its own function-calling traffic: a vocabulary of
made-up names (fn_<k>, p_<k>, v_<k>), a toy tokenizer (structural characters are single tokens,
identifiers and string contents are cut into pieces of at most four characters) and a small
JSON state machine that names the role of every emitted token.

Decode-side tag ids (generated tokens):
    0 required-key   1 enum-value   2 argument-value   3 boundary   4 scaffold   5 free-text
Prompt-side label ids:
    6 protected content   7 function name   8 parameter key   9 constraint   10 schema scaffold
TAG_PROTECTED (0xFF) marks tokens that are always kept at high precision.
"""
from __future__ import annotations

import numpy as np

from .rng import CounterRng

REQUIRED_KEY, ENUM_VALUE, ARGUMENT_VALUE, BOUNDARY, SCAFFOLD, FREE_TEXT = range(6)
P_PROTECTED, P_FUNCTION_NAME, P_PARAMETER_KEY, P_CONSTRAINT, P_SCHEMA_SCAFFOLD = range(6, 11)
TAG_PROTECTED = 0xFF
N_DECODE_TAGS = 6
N_ALL_TAGS = 11
TAG_NAMES = ["required-key", "enum-value", "argument-value", "boundary", "scaffold", "free-text",
             "protected-content", "function-name", "parameter-key", "constraint", "schema-scaffold"]

_TYPES = ["string", "integer", "number", "boolean", "enum"]
_SYLL = ["ka", "lo", "mi", "ru", "ta", "ne", "so", "vi", "du", "pe", "ga", "zu"]


def _pieces(text: str):
    """Toy tokenizer for identifier / string contents: pieces of at most four characters."""
    return [text[i:i + 4] for i in range(0, len(text), 4)]


class _Emitter:
    def __init__(self):
        self.tags = []

    def tok(self, tag: int, n: int = 1):
        self.tags.extend([tag] * n)

    def text(self, tag: int, s: str):
        self.tags.extend([tag] * len(_pieces(s)))

    def __len__(self):
        return len(self.tags)


def _word(rng: CounterRng, lo=2, hi=5) -> str:
    return "".join(rng.choice(_SYLL) for _ in range(rng.randint(lo, hi)))


def _make_tool(rng: CounterRng, k: int):
    """A made-up tool: name, parameters with type / required flag / enum domain."""
    n_params = rng.randint(1, 8)
    params = []
    for j in range(n_params):
        ty = _TYPES[rng.weighted([4, 2, 2, 1, 2])]
        params.append({
            "key": f"p_{rng.below(200)}_{_word(rng, 1, 2)}",
            "type": ty,
            "required": rng.unit() < 0.55 or j == 0,
            "enum": [f"v_{rng.below(500)}{_word(rng, 1, 2)}" for _ in range(rng.randint(2, 6))] if ty == "enum" else None,
        })
    return {"name": f"fn_{k}_{_word(rng, 1, 3)}", "params": params}


def _emit_value(em: _Emitter, rng: CounterRng, p):
    ty = p["type"]
    if ty == "enum":
        em.tok(SCAFFOLD)                      # opening quote
        em.text(ENUM_VALUE, rng.choice(p["enum"]))
        em.tok(SCAFFOLD)                      # closing quote
    elif ty == "string":
        em.tok(SCAFFOLD)
        if rng.unit() < 0.3:                  # long string contents read as free text
            s = " ".join(_word(rng, 1, 3) for _ in range(rng.randint(8, 40)))
            em.text(FREE_TEXT, s)
        else:
            em.text(ARGUMENT_VALUE, f"v_{rng.below(1000)}{_word(rng, 1, 3)}")
        em.tok(SCAFFOLD)
    elif ty == "integer":
        em.text(ARGUMENT_VALUE, str(rng.below(10 ** rng.randint(1, 7))))
    elif ty == "number":
        em.text(ARGUMENT_VALUE, f"{rng.below(10000)}.{rng.below(1000)}")
    else:
        em.tok(ARGUMENT_VALUE)                # true / false


def _emit_call(em: _Emitter, rng: CounterRng, tool):
    em.tok(BOUNDARY)                          # {
    for fixed in ("name",):
        em.tok(SCAFFOLD)                      # "
        em.text(SCAFFOLD, fixed)
        em.tok(SCAFFOLD, 3)                   # " : space
    em.tok(SCAFFOLD)                          # "
    em.text(ENUM_VALUE, tool["name"])         # the function is chosen from a legal set
    em.tok(SCAFFOLD, 3)                       # " , space
    em.tok(SCAFFOLD)
    em.text(SCAFFOLD, "arguments")
    em.tok(SCAFFOLD, 3)
    em.tok(BOUNDARY)                          # {
    first = True
    for p in tool["params"]:
        if not p["required"] and rng.unit() < 0.5:
            continue
        if not first:
            em.tok(SCAFFOLD, 2)               # , space
        first = False
        em.tok(SCAFFOLD)                      # "
        em.text(REQUIRED_KEY if p["required"] else SCAFFOLD, p["key"])
        em.tok(SCAFFOLD, 3)                   # " : space
        _emit_value(em, rng, p)
    em.tok(BOUNDARY, 2)                       # } }


def grammar_decode_tags(seed: int, seq: int, n_tokens: int) -> np.ndarray:
    """Tags of n_tokens generated tokens: turns of 1-4 synthetic function calls, concatenated."""
    rng = CounterRng(seed, 101, seq)
    tools = [_make_tool(rng, k) for k in range(rng.randint(3, 10))]
    em = _Emitter()
    while len(em) < n_tokens:
        if rng.unit() < 0.4:                  # optional preamble before the calls
            em.text(FREE_TEXT, " ".join(_word(rng, 1, 3) for _ in range(rng.randint(4, 30))))
        n_calls = 1 + rng.weighted([4, 3, 2, 1])
        em.tok(BOUNDARY)                      # [
        for c in range(n_calls):
            if c:
                em.tok(BOUNDARY)              # call separator
                em.tok(SCAFFOLD)
            _emit_call(em, rng, rng.choice(tools))
        em.tok(BOUNDARY, 2)                   # ] end-of-turn
    return np.asarray(em.tags[:n_tokens], dtype=np.uint8)


def grammar_prompt_tags(seed: int, seq: int, n_tokens: int) -> np.ndarray:
    """Labels of n_tokens prompt tokens: instructions, a synthetic tool schema, the user request."""
    rng = CounterRng(seed, 202, seq)
    em = _Emitter()
    n_head = max(1, int(n_tokens * 0.04))
    n_tail = max(1, int(n_tokens * 0.06))
    em.tok(P_PROTECTED, n_head)               # system instructions
    body = n_tokens - n_head - n_tail
    k = 0
    while len(em) < n_head + body:
        tool = _make_tool(rng, k)
        k += 1
        em.tok(P_SCHEMA_SCAFFOLD, 2)          # { "
        em.text(P_SCHEMA_SCAFFOLD, "name")
        em.tok(P_SCHEMA_SCAFFOLD, 3)
        em.text(P_FUNCTION_NAME, tool["name"])
        em.tok(P_SCHEMA_SCAFFOLD, 3)
        em.text(P_SCHEMA_SCAFFOLD, "description")
        em.tok(P_SCHEMA_SCAFFOLD, 3)
        em.text(P_SCHEMA_SCAFFOLD, " ".join(_word(rng, 1, 3) for _ in range(rng.randint(5, 25))))
        em.tok(P_SCHEMA_SCAFFOLD, 3)
        em.text(P_SCHEMA_SCAFFOLD, "parameters")
        em.tok(P_SCHEMA_SCAFFOLD, 4)
        em.text(P_SCHEMA_SCAFFOLD, "properties")
        em.tok(P_SCHEMA_SCAFFOLD, 3)
        for p in tool["params"]:
            em.tok(P_SCHEMA_SCAFFOLD)
            em.text(P_PARAMETER_KEY, p["key"])
            em.tok(P_SCHEMA_SCAFFOLD, 4)
            em.text(P_SCHEMA_SCAFFOLD, "type")
            em.tok(P_SCHEMA_SCAFFOLD, 3)
            em.text(P_CONSTRAINT, p["type"])
            em.tok(P_SCHEMA_SCAFFOLD, 2)
            if p["enum"]:
                em.text(P_SCHEMA_SCAFFOLD, "enum")
                em.tok(P_SCHEMA_SCAFFOLD, 3)
                for v in p["enum"]:
                    em.tok(P_SCHEMA_SCAFFOLD)
                    em.text(P_CONSTRAINT, v)
                    em.tok(P_SCHEMA_SCAFFOLD, 2)
                em.tok(P_SCHEMA_SCAFFOLD)
            elif p["type"] in ("integer", "number") and rng.unit() < 0.5:
                em.text(P_SCHEMA_SCAFFOLD, "minimum")
                em.tok(P_SCHEMA_SCAFFOLD, 2)
                em.text(P_CONSTRAINT, str(rng.below(100)))
                em.tok(P_SCHEMA_SCAFFOLD)
            em.text(P_SCHEMA_SCAFFOLD, "description")
            em.tok(P_SCHEMA_SCAFFOLD, 3)
            em.text(P_SCHEMA_SCAFFOLD, " ".join(_word(rng, 1, 3) for _ in range(rng.randint(3, 12))))
            em.tok(P_SCHEMA_SCAFFOLD, 3)
        em.tok(P_SCHEMA_SCAFFOLD, 2)
        em.text(P_SCHEMA_SCAFFOLD, "required")
        em.tok(P_SCHEMA_SCAFFOLD, 3)
        for p in tool["params"]:
            if p["required"]:
                em.tok(P_SCHEMA_SCAFFOLD)
                em.text(P_CONSTRAINT, p["key"])
                em.tok(P_SCHEMA_SCAFFOLD, 2)
        em.tok(P_SCHEMA_SCAFFOLD, 4)
    tags = em.tags[:n_head + body] + [P_PROTECTED] * n_tail   # the user's request closes the prompt
    return np.asarray(tags[:n_tokens], dtype=np.uint8)


def mix_tags(seed: int, seq: int, n_tokens: int, tag_ids, probs, mean_run: float = 3.0,
             stream: int = 303) -> np.ndarray:
    """Run-structured stream with a target stationary mix: each run draws its tag from `probs`
    and a geometric length with the given mean."""
    rng = CounterRng(seed, stream, seq)
    out = np.empty(n_tokens, dtype=np.uint8)
    i = 0
    p_stop = 1.0 / mean_run
    while i < n_tokens:
        tag = tag_ids[rng.weighted(probs)]
        run = 1
        while rng.unit() >= p_stop:
            run += 1
        out[i:i + run] = tag
        i += run
    return out


def mix_decode_tags(seed: int, seq: int, n_tokens: int) -> np.ndarray:
    """Scaffold/boundary-heavy decode stream: 45 % scaffold, 25 % boundary, 7.5 % each other tag."""
    ids = [SCAFFOLD, BOUNDARY, REQUIRED_KEY, ENUM_VALUE, ARGUMENT_VALUE, FREE_TEXT]
    return mix_tags(seed, seq, n_tokens, ids, [0.45, 0.25, 0.075, 0.075, 0.075, 0.075])


def mix_prompt_tags(seed: int, seq: int, n_tokens: int) -> np.ndarray:
    ids = [P_SCHEMA_SCAFFOLD, P_PARAMETER_KEY, P_CONSTRAINT, P_FUNCTION_NAME, P_PROTECTED]
    return mix_tags(seed, seq, n_tokens, ids, [0.55, 0.15, 0.15, 0.05, 0.10], stream=404)


# ---- synthetic parser states -------------------------------------------------------------
# The online lookup also sees the parser state s_t (it selects the reserve and says whether the
# position is critical).  The toy grammar above has no automaton to take states from, so a state
# id is derived from the tag stream itself: which structural class the token belongs to and how
# far into a run of that class it sits (0, 1, 2, 3+).  Ids: tag * 4 + min(run position, 3) for
# the eleven table tags, 44 for protected tokens, 47 for anything else.
N_STATES = 48
STATE_PROTECTED = 44
STATE_OTHER = 47


def parser_states(tags: np.ndarray) -> np.ndarray:
    out = np.zeros(tags.shape[0], dtype=np.uint16)
    run = 0
    for i, z in enumerate(tags.tolist()):
        run = run + 1 if i and tags[i - 1] == z else 0
        if z < N_ALL_TAGS:
            out[i] = z * 4 + min(run, 3)
        else:
            out[i] = STATE_PROTECTED if z == TAG_PROTECTED else STATE_OTHER
    return out


def critical_states() -> np.ndarray:
    """Flags of the states treated as critical or lookahead-critical: everything inside a required
    key or an enum value, and the first token of an argument value or of a boundary."""
    crit = np.zeros(N_STATES, dtype=np.uint8)
    for z in (REQUIRED_KEY, ENUM_VALUE):
        crit[z * 4:z * 4 + 4] = 1
    crit[ARGUMENT_VALUE * 4] = 1
    crit[BOUNDARY * 4] = 1
    return crit
