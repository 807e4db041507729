"""Pins of the kernel-looping pass (paper_2410_23668_b200/looping_pass.py) against what the paper prints: the lattice
of Section 3.1, the usage-property sets, transformed kernels and merged calls of the four worked examples of
Section 3.3 (tests/golden/looping_examples.json), and the call counts of Section 2 for this package's own decode
step (tests/golden/call_counts.txt).  CPU only."""
import itertools
import json
from pathlib import Path

import pytest

from paper_2410_23668_b200 import looping_pass as lp

GOLDEN = json.loads((Path(__file__).parent / "golden" / "looping_examples.json").read_text())["examples"]
S = lp._s


# What the four example kernels compute, in this package's own IR statements: (a) accumulates a product into its
# third parameter, (b) writes a difference, (c) one matrix product per call, (d) the same product swept over row tiles.
BODIES = {
    "a": ["z = z + y * x"],
    "b": ["z = y - x"],
    "c": ["z = w * x"],
    "d": [("for (r = 0; r < M; r += R)", ["z[r::r+R] = w[r::r+R] * x"])],
}


def _example(name):
    g = GOLDEN[name]
    k = lp.kernel("kernel_" + name, list(g["param_shapes"].items()), BODIES[name])
    calls = [lp.Call(k.name, tuple(a)) for a in g["calls"]]
    return g, k, calls, set(g["live_after"])


def _flat(items):
    return [it.text if isinstance(it, lp.Stmt) else [it.header, _flat(it.body)] for it in items]


def _stored(stores):
    """Parameters a list of store statements writes (text before the first bracket or blank, prime dropped)."""
    return [st.split("[")[0].split(" ")[0].rstrip("'") for st in stores]


def test_lattice_is_the_papers():
    # fourteen elements; the numbered ones are exactly the seven sets the figure's caption calls well-defined
    assert len(set(lp.ELEMENTS)) == 14
    assert [lp.E1, lp.E2, lp.E3, lp.E4, lp.E5, lp.E6, lp.E7] == [
        S("Const", "In"), S("In", "Local"), S("In", "Live"), S("Local", "Out"), S("Live", "Out"),
        S("In", "Live", "Out"), S("Local", "Live", "Out")]
    # it is a lattice: every pair has exactly one least upper bound; the join is idempotent, commutative, associative
    for a, b in itertools.product(lp.ELEMENTS, repeat=2):
        j = lp.join(a, b)
        assert lp.leq(a, j) and lp.leq(b, j) and j == lp.join(b, a)
        assert lp.join(a, a) == a
    for a, b, c in itertools.product(lp.ELEMENTS, repeat=3):
        assert lp.join(lp.join(a, b), c) == lp.join(a, lp.join(b, c))
    # the order is set inclusion wherever both sides are sets, and everything lies below the top
    for a, b in itertools.product(lp.ELEMENTS[:-1], repeat=2):
        if lp.leq(a, b):
            assert a <= b
    assert all(lp.leq(e, lp.TOP) for e in lp.ELEMENTS)
    # "constrained" union: the union where it is one of the seven sets ...
    assert lp.join(S("In"), S("Local")) == lp.E2 and lp.join(S("Live"), S("Out")) == lp.E5
    assert lp.join(lp.E3, lp.E5) == lp.E6 and lp.join(lp.E4, lp.E5) == lp.E7 and lp.join(S("Const"), S("In")) == lp.E1
    # ... otherwise the next well-defined set above it, or the top (= no match)
    assert lp.join(S("In"), S("Out")) == lp.E6          # read and written: handled like a live in/out parameter
    assert lp.join(S("Local"), S("Live")) == lp.E7
    assert lp.join(S("Const"), S("Out")) == lp.TOP      # one tensor written by every call
    assert lp.join(lp.E1, S("Local")) == lp.TOP and lp.join(lp.E2, S("Out")) == lp.TOP and lp.join(lp.E6, lp.E7) == lp.TOP


@pytest.mark.parametrize("name", sorted(GOLDEN))
def test_worked_examples(name):
    g, k, calls, live = _example(name)
    u = lp.usage_properties(k, calls, live)
    assert {p: sorted(v) for p, v in u.P.items()} == {p: sorted(v) for p, v in g["P"].items()}
    assert u.match
    t = lp.transform(k, calls, live)
    assert t.name == k.name + "'" and t.n_calls == len(calls)
    assert dict(t.params) == g["shapes"]
    assert len(t.buffers) == g["n_buffers"]
    if t.buffers:
        assert t.buffers[0][2] == g["buffer_init"] and all(b[2] is None for b in t.buffers[1:])
    assert _stored(t.istores) == g["stored_in_loop"] and _stored(t.estores) == g["stored_after_loop"]
    # grouped parameters are indexed by the loop counter in the body, parameters kept in a buffer do not appear
    body_text = " ".join(str(x) for x in _flat(t.body))
    for prm, shape in g["shapes"].items():
        name = prm.rstrip("'")
        grouped = shape != g["param_shapes"][name]
        if grouped and name not in g["stored_in_loop"]:
            assert prm + "[n]" in body_text, (prm, body_text)
    assert [list(a) if isinstance(a, tuple) else a for a in t.args] == g["args"]
    text = t.render()
    assert text.splitlines()[0] == f"{k.name}'(" + ", ".join(f"{n}[{s}]" for n, s in g["shapes"].items()) + ")"
    assert f"for(n = 0; n < {len(calls)}; ++n)" in text


def test_what_breaks_a_chain():
    g, k, calls, live = _example("c")
    # the intermediate result is also read by another parameter of the next call: not uniquely chained
    k2 = lp.kernel("k2", [("w", "MxM"), ("x", "MxN"), ("z", "MxN")], ["z = w * x"])
    u = lp.usage_properties(k2, [lp.Call("k2", ("w0", "x", "y")), lp.Call("k2", ("y", "y", "z"))], {"z"})
    assert "Local" not in u.P["x"] and "Local" not in u.P["z"]
    # the writes do not cover what the next call reads (a loop over part of the rows): no promotion to a buffer
    kp = lp.kernel("kp", [("w", "MxM"), ("x", "MxN"), ("z", "MxN")],
                   [("for (t = 0; t < M / 2; t += T)", ["z[t::t+T] = w[t::t+T] * x"], False)])
    u = lp.usage_properties(kp, [lp.Call("kp", a) for a in (("w0", "x", "y"), ("w1", "y", "z"))], {"z"})
    assert u.P == {"w": S("In"), "x": S("In"), "z": S("Out")} and u.match and all(u.group(p) for p in u.P)
    # example (c) with the intermediate live afterwards: the chain stays, the store moves into the loop
    u = lp.usage_properties(k, calls, {"y", "z"})
    assert u.P["z"] == lp.E7
    t = lp.transform(k, calls, {"y", "z"})
    assert t.istores == ("z'[n] = buf",) and t.estores == () and dict(t.params)["z'"] == "2xMxN" and t.args[2] == ("y", "z")
    # one tensor passed to a written parameter in every call: the top element, no match, no transformation
    ka = lp.kernel("acc", [("x", "N"), ("z", "N")], ["z = x"])
    bad = [lp.Call("acc", ("a", "s")), lp.Call("acc", ("b", "s"))]
    u = lp.usage_properties(ka, bad, {"s"})
    assert u.P["z"] == lp.TOP and not u.match
    with pytest.raises(ValueError):
        lp.transform(ka, bad, {"s"})


def _decode_program(L):
    """The per-layer schedule of one decode step (Section 2, schedule (ii)) in the toy IR: embedding, L calls to the
    decoder-layer kernel chained through the hidden state, classifier, sampling."""
    layer = lp.kernel("decoder_layer", [("x_in", "H"), ("x_out", "H"), ("w", "S"), ("kv", "2xCxD"), ("pos", "1")],
                      ["kv[pos] = w * x_in", "x_out = x_in + w * kv"])
    kernels = {
        "embedding": lp.kernel("embedding", [("tok", "1"), ("e", "VxH"), ("x", "H")], ["x = e[tok]"]),
        "decoder_layer": layer,
        "classifier": lp.kernel("classifier", [("x", "H"), ("wlm", "VxH"), ("logits", "V")], ["logits = wlm * x"]),
        "sampling": lp.kernel("sampling", [("logits", "V"), ("next", "1")], ["next = logits"]),
    }
    calls = [lp.Call("embedding", ("tok", "E", "x0"))]
    calls += [lp.Call("decoder_layer", (f"x{l}", f"x{l + 1}", f"w{l}", f"kv{l}", "pos")) for l in range(L)]
    calls += [lp.Call("classifier", (f"x{L}", "Wlm", "logits")), lp.Call("sampling", ("logits", "next"))]
    outputs = frozenset({"next", "logits", f"x{L}"} | {f"kv{l}" for l in range(L)})
    return lp.Program(kernels, tuple(calls), outputs)


def test_decode_step_call_counts_and_argument_grouping():
    counts = {}
    for line in (Path(__file__).parent / "golden" / "call_counts.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            key, val = line.split("=")
            counts[key.strip()] = int(val)
    L = 32
    prog = _decode_program(L)
    assert len(prog.calls) == counts["per_layer_launches"]          # 35 calls per token
    sched = lp.loop_program(prog)
    assert len(sched) == counts["looped_launches"]                      # 4 calls per token
    looped = sched[1]
    assert isinstance(looped, lp.LoopedKernel) and looped.n_calls == L
    u = lp.usage_properties(prog.kernels["decoder_layer"], prog.calls[1:1 + L], prog.live_after(L))
    assert u.P == {"x_in": lp.E2, "x_out": lp.E4, "w": S("In"), "kv": lp.E6, "pos": lp.E1}
    # the merged call's arguments are the argument rule of kl_decode_step: the hidden state enters once (from the
    # embedding) and leaves once, weights and cache slices of all layers are grouped, the position is passed once
    assert looped.args[0] == "x0" and looped.args[1] == f"x{L}" and looped.args[4] == "pos"
    assert looped.args[2] == tuple(f"w{l}" for l in range(L)) and looped.args[3] == tuple(f"kv{l}" for l in range(L))
    assert dict(looped.params) == {"x_in'": "H", "x_out'": "H", "w'": f"{L}xS", "kv'": f"{L}x2xCxD", "pos'": "1"}
    assert looped.buffers == (("buf", "H", "x_in'"),) and looped.estores == ("x_out' = buf",) and looped.istores == ()
    assert [s.text for s in looped.body] == ["kv'[n][pos'] = w'[n] * buf", "buf = buf + w'[n] * kv'[n]"]
