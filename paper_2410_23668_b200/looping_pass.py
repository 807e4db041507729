"""Kernel looping as a compiler pass over a toy intermediate representation (Sections 3.1 - 3.3 of the paper).

The CUDA library in this package IS a kernel-looped decoder written by hand; this module is the analysis and the
rewrite that the paper describes for deriving such a kernel mechanically, on an IR just large enough to hold the
paper's worked examples and the decode step's own call sequence:

  * usage properties of a kernel parameter over N calls -- Const, In, Local, Live, Out (Section 3.1, the table of
    usage properties), from the parameter's arguments a[i][0..N-1], the kernel body's reads and writes, and the
    tensors live after the last call;
  * the lattice over sets of those properties (Section 3.1, the lattice figure): P(p) is the join of the properties
    that hold (Eq. 1); a list of calls matches when no parameter reaches the top element (Eq. 2);
  * Group(p) (Section 3.2, Eq. 3) and the rewrite rules (1) - (10) of the transformation figure: one kernel with a loop
    over the N calls, grouped parameters indexed by the loop counter, chained (Local) parameters kept in an on-chip
    buffer, stores back per iteration (Live) or once at the end, and the merged call's arguments.

The IR is textual on purpose.  A kernel body is a list of statements `lhs = rhs` / `lhs += rhs` whose operands are
parameter names with an optional subscript (`z[t::t+T]`), and `for` loops around such statements; reads and writes
are derived from the text.  Address-space coverage (the paper's WriteSpace >= ReadSpace, for which it points at
polyhedral analysis) is decided by the one rule such an IR supports: a whole-tensor write covers everything, and a
subscripted write inside a loop covers the tensor when the loop is declared a full sweep.

Nothing here is used by the decode path; tests pin it to the paper's four printed examples and apply it to the
per-layer call sequence of this package's own decoder, where it yields the argument grouping of kl_decode_step.
"""
from __future__ import annotations

import re
from dataclasses import dataclass

CONST, IN, LOCAL, LIVE, OUT = "Const", "In", "Local", "Live", "Out"
TOP = "TOP"   # the lattice's top element: a match failure


def _s(*names: str) -> frozenset:
    return frozenset(names)


# Elements of the lattice (Section 3.1): the empty set, the five singletons, the seven numbered sets, and the top.
E1, E2, E3, E4 = _s(CONST, IN), _s(IN, LOCAL), _s(IN, LIVE), _s(LOCAL, OUT)
E5, E6, E7 = _s(LIVE, OUT), _s(IN, LIVE, OUT), _s(LOCAL, LIVE, OUT)
ELEMENTS = (_s(), _s(CONST), _s(IN), _s(LOCAL), _s(LIVE), _s(OUT), E1, E2, E3, E4, E5, E6, E7, TOP)
# Hasse diagram, edges upward, as drawn in the paper's figure
COVERS = {
    _s(): (_s(CONST), _s(IN), _s(LOCAL), _s(LIVE), _s(OUT)),
    _s(CONST): (E1,),
    _s(IN): (E1, E2, E3),
    _s(OUT): (E4, E5),
    _s(LOCAL): (E2, E4),
    _s(LIVE): (E3, E5),
    E3: (E6,), E5: (E6, E7), E4: (E7,),
    E1: (TOP,), E2: (TOP,), E6: (TOP,), E7: (TOP,),
    TOP: (),
}


def _up(e) -> set:
    """All elements at or above e."""
    seen, todo = {e}, [e]
    while todo:
        for n in COVERS[todo.pop()]:
            if n not in seen:
                seen.add(n)
                todo.append(n)
    return seen


def leq(a, b) -> bool:
    return b in _up(a)


def join(a, b):
    """Least upper bound in the lattice (the paper's operator on property sets in Eq. 1)."""
    common = _up(a) & _up(b)
    least = [c for c in common if all(leq(c, d) for d in common)]
    assert len(least) == 1, (a, b, least)   # it is a lattice: checked for every pair by the tests
    return least[0]


# ------------------------------------------------------------------------------------------------ the IR

@dataclass(frozen=True)
class Ref:
    """One occurrence of a parameter in a statement."""
    param: str
    write: bool
    subscript: str   # "" for the whole tensor, else the text between the brackets


@dataclass(frozen=True)
class Stmt:
    text: str

    def refs(self, params) -> list[Ref]:
        m = re.match(r"^(.*?)(\+=|=)(.*)$", self.text)
        assert m, self.text
        lhs, op, rhs = m.group(1), m.group(2), m.group(3)
        out = []
        for side, is_lhs in ((lhs, True), (rhs, False)):
            for name, sub in _occurrences(side, params):
                if is_lhs:
                    out.append(Ref(name, True, sub))
                    if op == "+=":
                        out.append(Ref(name, False, sub))
                else:
                    out.append(Ref(name, False, sub))
                # parameters that appear inside a subscript are read, on either side
                out += [Ref(n2, False, s2) for n2, s2 in _occurrences(sub, params)]
        return out


@dataclass(frozen=True)
class Loop:
    header: str               # e.g. "for (t = 0; t < M; t += T)"
    body: tuple               # of Stmt / Loop
    full_sweep: bool = True   # subscripted writes in this loop cover the whole tensor over its iterations


@dataclass(frozen=True)
class Kernel:
    name: str
    params: tuple             # of (name, shape) with shape a string such as "N" or "MxN"
    body: tuple               # of Stmt / Loop

    @property
    def names(self) -> list[str]:
        return [n for n, _ in self.params]


@dataclass(frozen=True)
class Call:
    kernel: str
    args: tuple               # tensor names, one per parameter


def kernel(name: str, params, body) -> Kernel:
    """Convenience constructor: params [(name, shape)], body a nested list of strings and (header, [body]) pairs."""
    def conv(items):
        out = []
        for it in items:
            if isinstance(it, str):
                out.append(Stmt(it.strip()))
            else:
                out.append(Loop(it[0], conv(it[1]), it[2] if len(it) > 2 else True))
        return tuple(out)
    return Kernel(name, tuple(params), conv(body))


def _occurrences(text: str, params):
    """(name, subscript) of every parameter occurrence in text."""
    if not params:
        return []
    pat = re.compile(r"\b(" + "|".join(re.escape(p) for p in sorted(params, key=len, reverse=True)) + r")\b(?:\[([^\]]*)\])?")
    return [(m.group(1), m.group(2) or "") for m in pat.finditer(text)]


def _walk(body, covered=True):
    """Yields (statement, every enclosing loop is a full sweep)."""
    for it in body:
        if isinstance(it, Stmt):
            yield it, covered
        else:
            yield from _walk(it.body, covered and it.full_sweep)


# ------------------------------------------------------------------------------------------------ analysis (3.1)

def reads(k: Kernel) -> set:
    return {r.param for st, _ in _walk(k.body) for r in st.refs(k.names) if not r.write}


def writes(k: Kernel) -> set:
    return {r.param for st, _ in _walk(k.body) for r in st.refs(k.names) if r.write}


def write_covers_all(k: Kernel, p: str) -> bool:
    """WriteSpace(p) is the whole tensor: a whole-tensor write, or subscripted writes under full-sweep loops only."""
    ws = [(r, cov) for st, cov in _walk(k.body) for r in st.refs(k.names) if r.write and r.param == p]
    if not ws:
        return False
    return any(r.subscript == "" for r, _ in ws) or all(cov for _, cov in ws)


def written_in_parts(k: Kernel, p: str) -> bool:
    return any(r.write and r.param == p and r.subscript != "" for st, _ in _walk(k.body) for r in st.refs(k.names))


@dataclass(frozen=True)
class Usage:
    """Result of the analysis for one list of calls."""
    P: dict            # parameter -> frozenset of properties, or TOP
    partner: dict      # Local parameter -> the parameter it is chained with
    n_calls: int

    @property
    def match(self) -> bool:   # Eq. 2
        return all(v != TOP for v in self.P.values())

    def group(self, p: str) -> bool:   # Eq. 3
        s = self.P[p]
        return LIVE in s or (LOCAL not in s and CONST not in s)


def usage_properties(k: Kernel, calls, live_after) -> Usage:
    """Usage properties of every parameter of k over the calls c_0 .. c_{N-1} (all calls to k), given the tensors that
    are live after c_{N-1}.  Argument a[i][n] is the tensor passed for parameter i in call n."""
    names, N = k.names, len(calls)
    assert N >= 1 and all(c.kernel == k.name and len(c.args) == len(names) for c in calls)
    a = {p: [c.args[i] for c in calls] for i, p in enumerate(names)}
    rd, wr = reads(k), writes(k)

    def chained(src: str, dst: str) -> bool:   # what src holds after call n is what dst gets in call n + 1, for every n
        return N >= 2 and all(a[src][n] == a[dst][n + 1] for n in range(N - 1))

    # Local comes in pairs: a written parameter j whose every result is read by exactly one parameter i of the next
    # call, by nobody else in that call, and whose writes cover everything i reads
    partner = {}
    for j in names:
        if j not in wr:
            continue
        readers = [i for i in names if i != j and i in rd and chained(j, i)]
        if len(readers) != 1:
            continue
        i = readers[0]
        writers = [h for h in names if h != i and h in wr and chained(h, i)]
        if writers != [j]:
            continue
        others = any(a[j][n] == a[h][n + 1] for n in range(N - 1) for h in names if h != i)
        if others or not write_covers_all(k, j):
            continue
        partner[i], partner[j] = j, i

    P = {}
    for p in names:
        props = []
        if len(set(a[p])) == 1:
            props.append(CONST)
        if p in rd:
            props.append(IN)
        if p in partner:
            props.append(LOCAL)
        if p in wr and any(a[p][n] in live_after for n in range(N - 1)):
            props.append(LIVE)
        if p in wr:
            props.append(OUT)
        e = _s()
        for f in props:   # Eq. 1: the join of the singleton sets of the properties that hold
            e = join(e, _s(f))
        P[p] = e
    return Usage(P, partner, N)


# ------------------------------------------------------------------------------------------------ transformation (3.2)

@dataclass(frozen=True)
class LoopedKernel:
    """The kernel after rules (1) - (10), and the arguments of the single call that replaces the N calls."""
    name: str
    params: tuple        # (name', shape'), rule (2)
    buffers: tuple       # (buffer, shape, initialised from or None): on-chip, rules (3) - (4)
    n_calls: int
    body: tuple          # statements / loops of one iteration, references rewritten by rule (6)
    istores: tuple       # at the end of every iteration, rule (8)
    estores: tuple       # once after the loop, rule (10)
    args: tuple          # per parameter: one tensor name, or the tuple of all N arguments for a grouped parameter

    def render(self) -> str:
        """The transformed kernel as text, in the style of the paper's examples."""
        out = [f"{self.name}({', '.join(f'{n}[{s}]' for n, s in self.params)})"]
        for b, shape, init in self.buffers:
            out.append(f"  @onchip {b}[{shape}]" + (f" = {init}" if init else ""))
        out.append(f"  for(n = 0; n < {self.n_calls}; ++n)")

        def emit(items, depth):
            for it in items:
                if isinstance(it, Stmt):
                    out.append("  " * depth + it.text)
                else:
                    out.append("  " * depth + it.header)
                    emit(it.body, depth + 1)
        emit(self.body, 2)
        out += ["    " + t for t in self.istores] + ["  " + t for t in self.estores]
        return "\n".join(out)


def transform(k: Kernel, calls, live_after) -> LoopedKernel:
    """Rules (1) - (10) of Section 3.2 for a matched list of calls.  Raises ValueError when the calls do not match."""
    u = usage_properties(k, calls, live_after)
    if not u.match:
        raise ValueError("no match: " + ", ".join(p for p, v in u.P.items() if v == TOP) + " reached the top element")
    N, names = u.n_calls, k.names
    prime = {p: p + "'" for p in names}
    # rule (2): grouped parameters gain an outermost dimension N
    params = tuple((prime[p], f"{N}x{s}" if u.group(p) else s) for p, s in k.params)
    # rules (3), (4): one on-chip buffer per Local pair, initialised from the read parameter.  When the written
    # parameter is produced in parts while the read one may still be needed, the pair gets two buffers that swap at
    # the end of every iteration (the paper elides the test; this is the one its tiled example calls for).
    rbuf, wbuf, buffers, swaps = {}, {}, [], []
    pairs = [(i, u.partner[i]) for i in names if u.P[i] == E2]
    for idx, (i, j) in enumerate(pairs):
        tag = "" if len(pairs) == 1 else str(idx)
        shape = dict(k.params)[i]
        if written_in_parts(k, j):
            b0, b1 = f"buf{tag}0" if tag else "buf0", f"buf{tag}1" if tag else "buf1"
            buffers += [(b0, shape, prime[i]), (b1, shape, None)]
            rbuf[i], wbuf[j] = b0, b1
            swaps.append(f"{b0} = {b1}")
        else:
            b = f"buf{tag}"
            buffers.append((b, shape, prime[i]))
            rbuf[i], wbuf[j] = b, b

    # rules (5), (6): every reference becomes the buffer (Local), p'[n] (grouped) or p' (otherwise)
    pat = re.compile(r"\b(" + "|".join(re.escape(p) for p in sorted(names, key=len, reverse=True)) + r")\b(\[[^\]]*\])?")

    def rewrite(text: str) -> str:
        def sub(m):
            p, idx = m.group(1), m.group(2) or ""
            if idx:
                idx = "[" + rewrite(idx[1:-1]) + "]"
            if p in rbuf or p in wbuf:
                return (rbuf.get(p) or wbuf.get(p)) + idx
            return prime[p] + ("[n]" if u.group(p) else "") + idx
        return pat.sub(sub, text)

    def conv(items):
        return tuple(Stmt(rewrite(it.text)) if isinstance(it, Stmt) else Loop(it.header, conv(it.body), it.full_sweep)
                     for it in items)
    body = conv(k.body) + tuple(Stmt(t) for t in swaps)
    # rules (7) - (10): stores from the buffers back to their output parameters
    istores = tuple(f"{prime[p]}[n] = {wbuf[p]}" for p in names if u.P[p] == E7)
    estores = tuple(f"{prime[p]} = {wbuf[p]}" for p in names if u.P[p] == E4)
    # the merged call: Const -> its one argument, {In, Local} -> the first, {Local, Out} -> the last, grouped -> all
    args = []
    for i, p in enumerate(names):
        a = [c.args[i] for c in calls]
        if u.group(p):
            args.append(tuple(a))
        elif u.P[p] == E2:
            args.append(a[0])
        elif u.P[p] == E4:
            args.append(a[-1])
        else:   # Const
            args.append(a[0])
    return LoopedKernel(k.name + "'", params, tuple(buffers), N, body, istores, estores, tuple(args))


# ------------------------------------------------------------------------------------------------ over a program

@dataclass(frozen=True)
class Program:
    kernels: dict        # name -> Kernel
    calls: tuple         # of Call, in program order
    outputs: frozenset   # tensors the program's caller reads afterwards

    def live_after(self, idx: int) -> set:
        """Tensors read by a call after calls[idx], or by the caller."""
        live = set(self.outputs)
        for c in self.calls[idx + 1:]:
            k = self.kernels[c.kernel]
            rd = reads(k)
            live |= {arg for p, arg in zip(k.names, c.args) if p in rd}
        return live


def loop_program(prog: Program, min_calls: int = 2):
    """The greedy pass of Section 3.1: scans the call list and replaces every longest run of at least `min_calls`
    consecutive calls to one kernel that matches by its looped form.  Returns the new schedule, a list whose items
    are either the original Call or a LoopedKernel."""
    out, i, n = [], 0, len(prog.calls)
    while i < n:
        k = prog.kernels[prog.calls[i].kernel]
        j = i
        while j + 1 < n and prog.calls[j + 1].kernel == k.name:
            j += 1
        best = None
        for end in range(j, i + min_calls - 2, -1):   # longest first
            run = prog.calls[i:end + 1]
            if len(run) >= min_calls and usage_properties(k, run, prog.live_after(end)).match:
                best = end
                break
        if best is None:
            out.append(prog.calls[i])
            i += 1
        else:
            out.append(transform(k, prog.calls[i:best + 1], prog.live_after(best)))
            i = best + 1
    return out
