"""Reader of tests/golden/alg2_trace.txt: the hand-made 16-vertex index and the hand-worked run of
Alg. 2 on it.  Returns plain numpy arrays in the index layout (vectors in rank order, padded to 4
floats; ENC as [n, H, m] ranks with 0xFFFFFFFF for an empty entry) and the expected trace."""
import os

import numpy as np

PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "alg2_trace.txt")
BOT = 0xFFFFFFFF


def load():
    g = {"exp": []}
    vec, enc = {}, {}
    with open(PATH) as f:
        for ln in f:
            ln = ln.strip()
            if not ln or ln.startswith("#"):
                continue
            key, rest = ln.split(None, 1)
            if key == "vec":
                r, x, y = map(int, rest.split())
                vec[r] = (x, y)
            elif key == "enc":
                u, rows = rest.split(":")
                enc[int(u)] = [[BOT if t == "." else int(t) for t in row.split()] for row in rows.split("|")]
            elif key == "exp":
                _, body = rest.split(":", 1)
                u, en, pool = body.split("|")
                pool = [tuple(map(int, t.split(":"))) for t in pool.split()]
                g["exp"].append(dict(u=int(u), en=[int(t) for t in en.split()], pool=pool))
            else:
                vals = [int(t) for t in rest.split()]
                g[key] = vals[0] if len(vals) == 1 and key not in ("entry_points",) else vals
    n, H, m, d = g["n"], g["H"], g["m"], g["d"]
    assert sorted(vec) == list(range(n)) and sorted(enc) == list(range(n))
    d_pad = 4 * ((d + 3) // 4)
    V = np.zeros((n, d_pad), dtype=np.float32)
    for r, xy in vec.items():
        V[r, :d] = xy
    E = np.empty((n, H, m), dtype=np.uint32)
    for u, rows in enc.items():
        assert len(rows) == H and all(len(r) == m for r in rows)
        E[u] = np.array(rows, dtype=np.uint32)
    g.update(vectors=V, enc=E, d_pad=d_pad,
             sorted_attr=(10 * np.arange(n)).astype(np.int32),
             rank2id=((7 * np.arange(n) + 3) % n).astype(np.int32),
             query=np.zeros((1, d), dtype=np.float32))
    return g
