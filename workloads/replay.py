"""Replay an explicit operator list on a backend (harness code, no operator arithmetic).

A backend is any object with these methods (status 0 = success, negative = error;
a failing operator must leave the backend unchanged):

    payload(seed, stream, n)          -> backend-native transfer buffer of n tokens, filled by workloads.fill
    imp(buf, n)                       -> (status, ctx)
    materialize(ctx, t0, t1)          -> (status, buf)
    fork(ctx, k)                      -> (status, [ctx])
    append(ctxs, n_new, bufs)         -> (status, None)
    compose(ctxs, flags)              -> (status, ctx)
    evict(ctxs)                       -> (status, None)

``replay`` is a generator: it yields ``(index, op, status, result, names)`` after each
operator so that two backends can be stepped side by side with ``zip`` and compared.
"""
from __future__ import annotations


def replay(ops, backend, seed: int):
    names: dict[str, int] = {}
    bufs: dict[str, tuple] = {}
    for i, op in enumerate(ops):
        kind = op["op"]
        status, result = 0, None
        if kind == "import":
            buf = backend.payload(seed, op["stream"], op["n"])
            status, result = backend.imp(buf, op["n"])
            if status == 0:
                names[op["out"]] = result
        elif kind == "import_buf":
            buf, n = bufs[op["buf"]]
            status, result = backend.imp(buf, n)
            if status == 0:
                names[op["out"]] = result
        elif kind == "materialize":
            status, result = backend.materialize(names[op["ctx"]], op["t0"], op["t1"])
            if status == 0:
                bufs[op["out_buf"]] = (result, op["t1"] - op["t0"])
        elif kind == "drop_buf":
            bufs.pop(op["buf"], None)
        elif kind == "fork":
            status, result = backend.fork(names[op["ctx"]], op["k"])
            if status == 0:
                for nm, c in zip(op["out"], result):
                    names[nm] = c
        elif kind == "append":
            payloads = [backend.payload(seed, s, n) for s, n in zip(op["streams"], op["n_new"])]
            status, result = backend.append([names[c] for c in op["ctxs"]], list(op["n_new"]), payloads)
        elif kind == "compose":
            status, result = backend.compose([names[c] for c in op["segs"]], op.get("flags", 0))
            if status == 0:
                names[op["out"]] = result
        elif kind == "evict":
            status, result = backend.evict([names[c] for c in op["ctxs"]])
            if status == 0:
                for c in op["ctxs"]:
                    names.pop(c, None)
        else:
            raise ValueError(f"unknown op {kind!r}")
        yield i, op, status, result, dict(names)
