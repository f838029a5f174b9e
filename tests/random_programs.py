"""Seeded random tagged-Datalog programs inside the plan shapes the CUDA engine supports, for differential tests
against the oracle.  Plain data only (relations, rules, arrays): nothing here evaluates a rule."""
import numpy as np

from paper_2609_27203_b200 import workloads as W

V, Var, Atom, Rule, Const = W.V, W.Var, W.Atom, W.Rule, W.Const


def _edb(rng, dom, arity, n, sr):
    cols = [rng.integers(0, dom, n).astype(np.int32) for _ in range(arity)]
    if sr == W.MAXPLUS:
        tags = -rng.uniform(0.01, 0.7, n)           # log-probabilities: every cycle loses
    elif sr == W.MINPLUS:
        tags = rng.uniform(1.0, 10.0, n)            # positive lengths: every cycle costs
    elif sr == W.LOGSUMEXP:
        tags = rng.normal(0.0, 1.0, n)
    else:
        tags = rng.uniform(0.5, 1.5, n)
    return cols, tags.astype(np.float32)


def random_program(seed: int, dom: int = 0) -> W.Program:
    """dom = 0: the domain size is drawn from {5, 17, 60, 250}; otherwise it is `dom` (relations grow with it)."""
    rng = np.random.default_rng(seed)
    drawn = int(rng.choice([5, 17, 60, 250]))
    dom = dom or drawn
    sr = str(rng.choice([W.MAXPLUS, W.MINPLUS]))
    n_e = int(rng.integers(0, 5 * dom)) if rng.random() > 0.05 else 0
    n_f = int(rng.integers(1, 3 * dom))
    rels = {"e": (2, sr), "f": (2, sr)}
    facts = {"e": _edb(rng, dom, 2, n_e, sr), "f": _edb(rng, dom, 2, n_f, sr)}
    rules, outputs = [], []
    shape = int(rng.integers(0, 9))
    if shape == 0:      # left-linear closure, possibly with the edge probed on its second column and a second base rule
        rels["p"] = (2, sr)
        rules.append(Rule("p", (V(0), V(1)), (Atom("e", (Var(0), Var(1))),)))
        if rng.random() < 0.4:
            rules.append(Rule("p", (V(1), V(0)), (Atom("f", (Var(0), Var(1))),)))
        step = Atom("e", (Var(1), Var(2))) if rng.random() < 0.6 else Atom("f", (Var(2), Var(1)))
        rules.append(Rule("p", (V(0), V(2)), (Atom("p", (Var(0), Var(1))), step)))
        outputs.append("p")
    elif shape == 1:    # right-linear
        rels["p"] = (2, sr)
        rules.append(Rule("p", (V(0), V(1)), (Atom("e", (Var(0), Var(1))),)))
        rules.append(Rule("p", (V(0), V(2)), (Atom("e", (Var(0), Var(1))), Atom("p", (Var(1), Var(2))))))
        outputs.append("p")
    elif shape == 2:    # non-linear, with loaded facts in the derived relation
        rels["p"] = (2, sr)
        facts["p"] = _edb(rng, dom, 2, int(rng.integers(0, dom)), sr)
        rules.append(Rule("p", (V(0), V(1)), (Atom("e", (Var(0), Var(1))),)))
        rules.append(Rule("p", (V(0), V(2)), (Atom("p", (Var(0), Var(1))), Atom("p", (Var(1), Var(2))))))
        outputs.append("p")
    elif shape == 3:    # mutual recursion over two edge relations
        rels["p"] = (2, sr); rels["q"] = (2, sr)
        rules.append(Rule("p", (V(0), V(1)), (Atom("e", (Var(0), Var(1))),)))
        rules.append(Rule("q", (V(0), V(2)), (Atom("p", (Var(0), Var(1))), Atom("f", (Var(1), Var(2))))))
        rules.append(Rule("p", (V(0), V(2)), (Atom("q", (Var(0), Var(1))), Atom("e", (Var(1), Var(2))))))
        outputs += ["p", "q"]
    elif shape == 4:    # unary reachability from loaded seeds, two step rules into one head
        rels["r"] = (1, sr)
        k = int(rng.integers(1, 4))
        facts["r"] = ([rng.integers(0, dom, k).astype(np.int32)], _edb(rng, dom, 1, k, sr)[1])
        rules.append(Rule("r", (V(1),), (Atom("r", (Var(0),)), Atom("e", (Var(0), Var(1))))))
        if rng.random() < 0.5:
            rules.append(Rule("r", (V(1),), (Atom("r", (Var(0),)), Atom("f", (Var(1), Var(0))))))
        outputs.append("r")
    elif shape == 5:    # multi-source reachability: the source column is carried along
        rels["src"] = (1, sr); rels["reach"] = (2, sr)
        k = int(rng.integers(1, min(dom, 40) + 1))
        s = rng.choice(dom, k, replace=False).astype(np.int32)
        facts["src"] = ([s], np.zeros(k, np.float32))
        rules.append(Rule("reach", (V(0), V(0)), (Atom("src", (Var(0),)),)))
        rules.append(Rule("reach", (V(0), V(2)), (Atom("reach", (Var(0), Var(1))), Atom("e", (Var(1), Var(2))))))
        outputs.append("reach")
    elif shape == 6:    # a constant and a repeated variable on the scanned atom, then recursion on the result
        rels["h"] = (1, sr); rels["loop"] = (1, sr)
        c = int(rng.integers(0, dom))
        rules.append(Rule("h", (V(0),), (Atom("e", (Const(c), Var(0))),)))
        rules.append(Rule("h", (V(1),), (Atom("h", (Var(0),)), Atom("f", (Var(0), Var(1))))))
        rules.append(Rule("loop", (V(0),), (Atom("e", (Var(0), Var(0))),)))
        outputs += ["h", "loop"]
    elif shape == 7:    # closure, then negation over the finished relation and a plain join of two derived relations
        rels["p"] = (2, sr); rels["n"] = (2, sr); rels["j"] = (2, sr)
        rules.append(Rule("p", (V(0), V(1)), (Atom("e", (Var(0), Var(1))),)))
        rules.append(Rule("p", (V(0), V(2)), (Atom("p", (Var(0), Var(1))), Atom("e", (Var(1), Var(2))))))
        rules.append(Rule("n", (V(0), V(1)), (Atom("f", (Var(0), Var(1))), Atom("p", (Var(1), Var(2)), negated=True))))
        rules.append(Rule("j", (V(0), V(2)), (Atom("n", (Var(0), Var(1))), Atom("p", (Var(1), Var(2))))))
        outputs += ["p", "n", "j"]
    else:               # the cyclic joins over e and f
        rels["tri"] = (3, sr); rels["c4"] = (4, sr)
        rules.append(Rule("tri", (V(0), V(1), V(2)), (Atom("e", (Var(0), Var(1))), Atom("f", (Var(1), Var(2))), Atom("e", (Var(2), Var(0))))))
        rules.append(Rule("c4", (V(0), V(1), V(2), V(3)),
                          (Atom("e", (Var(0), Var(1))), Atom("f", (Var(1), Var(2))), Atom("f", (Var(2), Var(3))), Atom("e", (Var(3), Var(0))))))
        outputs += ["tri", "c4"]
    # a non-recursive aggregate stratum on its own relations
    agg = int(rng.integers(0, 8))
    if agg == 0:
        rels["a"] = (2, W.LOGSUMEXP); rels["b"] = (2, W.LOGSUMEXP); rels["s"] = (2, W.LOGSUMEXP)
        facts["a"] = _edb(rng, dom, 2, int(rng.integers(1, 4 * dom)), W.LOGSUMEXP)
        facts["b"] = _edb(rng, dom, 2, int(rng.integers(1, 4 * dom)), W.LOGSUMEXP)
        rules.append(Rule("s", (V(0), V(2)), (Atom("a", (Var(0), Var(1))), Atom("b", (Var(1), Var(2))))))
        outputs.append("s")
    elif agg == 1:
        rels["c"] = (2, W.SUMPROD); rels["deg"] = (2, W.SUMPROD)
        facts["c"] = _edb(rng, dom, 2, int(rng.integers(1, 4 * dom)), W.SUMPROD)
        rules.append(Rule("deg", (V(0),), (Atom("c", (Var(0), Var(1))),), emit_count=True))
        outputs.append("deg")
    elif agg == 2:      # two rules and loaded facts into one logsumexp head
        rels["a"] = (2, W.LOGSUMEXP); rels["b"] = (2, W.LOGSUMEXP); rels["s"] = (2, W.LOGSUMEXP)
        facts["a"] = _edb(rng, dom, 2, int(rng.integers(1, 4 * dom)), W.LOGSUMEXP)
        facts["b"] = _edb(rng, dom, 2, int(rng.integers(1, 4 * dom)), W.LOGSUMEXP)
        facts["s"] = _edb(rng, dom, 2, int(rng.integers(0, dom)), W.LOGSUMEXP)
        rules.append(Rule("s", (V(0), V(2)), (Atom("a", (Var(0), Var(1))), Atom("b", (Var(1), Var(2))))))
        rules.append(Rule("s", (V(1), V(0)), (Atom("a", (Var(0), Var(1))),)))
        outputs.append("s")
    elif agg == 3:      # affine patterns on both atoms and an affine head column (the digit-sum shape)
        rels["d"] = (2, W.LOGSUMEXP); rels["t"] = (2, W.LOGSUMEXP)
        n_img = 2 * int(rng.integers(1, 3 * dom))
        k = int(rng.integers(2, 11))
        img = np.repeat(np.arange(n_img, dtype=np.int32), k)
        dig = np.tile(np.arange(k, dtype=np.int32), n_img)
        keep = rng.random(len(img)) < 0.8
        facts["d"] = ([img[keep], dig[keep]], rng.normal(0, 1, int(keep.sum())).astype(np.float32))
        rules.append(Rule("t", (V(0), W.Affine(0, ((1, 1), (2, 1)))), (Atom("d", (Var(0, 2, 0), Var(1))), Atom("d", (Var(0, 2, 1), Var(2))))))
        outputs.append("t")
    elif agg == 4:      # a three-column relation: projected with a reduction, and looked up by its first column
        rels["g"] = (3, sr); rels["proj"] = (2, sr); rels["wide"] = (3, sr)
        facts["g"] = _edb(rng, dom, 3, int(rng.integers(1, 6 * dom)), sr)
        rules.append(Rule("proj", (V(0), V(2)), (Atom("g", (Var(0), Var(1), Var(2))),)))
        rules.append(Rule("wide", (V(0), V(2), V(3)), (Atom("f", (Var(0), Var(1))), Atom("g", (Var(1), Var(2), Var(3))))))
        outputs += ["proj", "wide"]
    elif agg == 5:      # two-step walk counts under sum-product, with a constant on the scanned atom in a second rule
        rels["c"] = (2, W.SUMPROD); rels["walk"] = (2, W.SUMPROD); rels["from0"] = (1, W.SUMPROD)
        facts["c"] = _edb(rng, dom, 2, int(rng.integers(1, 4 * dom)), W.SUMPROD)
        rules.append(Rule("walk", (V(0), V(2)), (Atom("c", (Var(0), Var(1))), Atom("c", (Var(1), Var(2))))))
        rules.append(Rule("from0", (V(1),), (Atom("c", (Const(int(rng.integers(0, dom))), Var(0))), Atom("c", (Var(0), Var(1))))))
        outputs += ["walk", "from0"]
    return W.Program(f"random_{seed}_shape{shape}_agg{agg}", rels, rules, facts, tuple(outputs))


def stretch(program: W.Program, stride: int, offset: int = 0) -> W.Program:
    """The same program with every stored value v replaced by v * stride + offset (and constants likewise): wide columns,
    64-bit packed keys.  Only for programs whose rules use plain variables and constants."""
    facts = {}
    for name, (cols, tags) in program.facts.items():
        facts[name] = ([(c.astype(np.int64) * stride + offset).astype(np.int32) for c in cols], tags)
    rules = []
    for r in program.rules:
        atoms = tuple(Atom(a.rel, tuple(Const(g.value * stride + offset) if isinstance(g, Const) else g for g in a.args), a.negated) for a in r.atoms)
        rules.append(Rule(r.head, r.head_exprs, atoms, r.emit_count))
    return W.Program(program.name + f"_x{stride}", dict(program.relations), rules, facts, program.outputs)
