"""Brute-force evaluation of a star-join query by full nested loops over
fact x dim_1 x ... x dim_J in pure Python.  Written independently of the
oracle (no hash maps, no shared helpers): it exists only to pin the oracle on
tiny inputs."""


def _holds(p, v):
    v = int(v)
    if p.op == "EQ":
        return v == p.lo
    if p.op == "NE":
        return v != p.lo
    if p.op == "LT":
        return v < p.lo
    if p.op == "LE":
        return v <= p.lo
    if p.op == "GT":
        return v > p.lo
    if p.op == "GE":
        return v >= p.lo
    if p.op == "BETWEEN":
        return p.lo <= v <= p.hi
    if p.op == "IN":
        return v in p.values
    raise ValueError(p.op)


def _wrap(x):
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


def _cmod(a, m):
    """C remainder: truncation toward zero."""
    q = abs(a) // abs(m)
    if (a < 0) != (m < 0):
        q = -q
    return a - q * m


def brute(w, fact, host_dims):
    """Returns ('DUP', None) or ('OK', {key: [sum, count]}) plus range flag."""
    n = len(next(iter(fact.values())))
    groups = {}
    out_of_range = False
    for i in range(n):
        if not all(_holds(p, fact[p.col][i]) for p in w.preds):
            continue
        matched = []
        alive = True
        for fk, dname in w.joins:
            spec = w.dim(dname)
            cols = host_dims[dname]
            hits = []
            for r in range(spec.rows):
                if int(cols[spec.key][r]) != int(fact[fk][i]):
                    continue
                if all(_holds(p, cols[p.col][r]) for p in spec.preds):
                    hits.append(r)
            if len(hits) > 1:
                return "DUP", None, False
            if not hits:
                alive = False
                break
            matched.append([int(cols[p][hits[0]]) for p in spec.payloads])
        if not alive:
            continue

        def term(t):
            raw = int(fact[t.a][i]) if t.src == "FACT" else matched[t.a][t.b]
            return _wrap(t.mult * raw)

        g = 0
        if w.mode != "SCALAR":
            g = w.key.offset
            for t in w.key.terms:
                g = _wrap(g + term(t))
            if w.key.modulo:
                g = _cmod(g, w.key.modulo)
            if w.mode == "DENSE" and not (0 <= g < w.num_groups):
                out_of_range = True
                continue
        v = term(w.agg.x)
        if w.agg.op == "MUL":
            v = _wrap(v * term(w.agg.y))
        elif w.agg.op == "SUB":
            v = _wrap(v - term(w.agg.y))
        elif w.agg.op == "ADD":
            v = _wrap(v + term(w.agg.y))
        s = groups.setdefault(g, [0, 0])
        s[0] = _wrap(s[0] + v)
        s[1] += 1
    return "OK", groups, out_of_range


def dup_keys_among_passing(spec, cols):
    seen = set()
    for r in range(spec.rows):
        if all(_holds(p, cols[p.col][r]) for p in spec.preds):
            k = int(cols[spec.key][r])
            if k in seen:
                return True
            seen.add(k)
    return False
