"""Writes block_d4.txt: one pre-norm decoder block (Eq. 5 with H(.) written out) on two tokens, multiplied out
with Python floats and `math` only.

Shape: hidden size 4, one query head and one KV head of dimension 4, MLP width 3, q/k/v biases, norm gains that
are not one, half-split rotation pairs (0, 2) and (1, 3), base 100, eps 1e-5.  The two tokens sit at global
positions 3 and 7 of a cache of 8 slots whose other slots hold zero keys and zero values: the row at position 3
sees slots 0..3 (three zero keys with logit 0 and its own), the row at position 7 sees all eight.  No oracle or array-library code is called.

Order of the block, as the Background and Attention Recovery sections give it for a pre-norm decoder:
  a  = x / sqrt(mean(x^2) + eps) * g_attn
  q  = R(m)(Wq a + bq),  k = R(m)(Wk a + bk),  v = Wv a + bv          (bias before the rotation)
  o  = sum_j softmax_j(q.k_j / sqrt(D)) v_j  over keys at positions <= m
  x1 = x + Wo o
  a2 = x1 / sqrt(mean(x1^2) + eps) * g_mlp
  x2 = x1 + Wd (silu(Wg a2) * (Wu a2)),  silu(t) = t / (1 + exp(-t))
"""
import math
import os

D = 4
F = 3
BASE = 100.0
EPS = 1e-5
POS = (3, 7)

X = [[0.5, -1.0, 0.25, 2.0], [-1.5, 0.75, 1.0, -0.25]]
G_ATTN = [1.5, 0.5, -1.0, 2.0]
G_MLP = [0.75, 1.25, 2.0, -0.5]
WQ = [[0.2, -0.1, 0.4, 0.3], [-0.3, 0.5, 0.1, -0.2], [0.6, 0.2, -0.4, 0.1], [0.1, -0.6, 0.3, 0.5]]
WK = [[-0.4, 0.3, 0.2, 0.1], [0.5, 0.1, -0.3, 0.4], [0.2, -0.5, 0.6, -0.1], [-0.1, 0.4, 0.3, -0.6]]
WV = [[0.3, 0.6, -0.2, 0.1], [-0.5, 0.2, 0.4, 0.3], [0.1, -0.3, 0.5, -0.4], [0.4, 0.1, -0.6, 0.2]]
WO = [[0.1, 0.4, -0.3, 0.2], [0.5, -0.2, 0.1, 0.6], [-0.4, 0.3, 0.2, -0.1], [0.2, 0.1, 0.5, -0.3]]
BQ = [0.3, -0.2, 0.1, 0.4]
BK = [-0.25, 0.5, 0.35, -0.15]
BV = [0.05, -0.1, 0.2, 0.3]
WG = [[0.4, -0.2, 0.1, 0.3], [-0.1, 0.5, 0.2, -0.4], [0.3, 0.1, -0.5, 0.2]]
WU = [[-0.3, 0.4, 0.2, 0.1], [0.2, 0.3, -0.1, 0.5], [0.6, -0.2, 0.4, -0.3]]
WD = [[0.2, -0.4, 0.1], [0.5, 0.3, -0.2], [-0.1, 0.6, 0.4], [0.3, -0.5, 0.2]]


def matvec(W, x):
    return [sum(W[r][c] * x[c] for c in range(len(x))) for r in range(len(W))]


def rms(x, g):
    ms = sum(t * t for t in x) / len(x)
    return [x[i] / math.sqrt(ms + EPS) * g[i] for i in range(len(x))]


def rotate(x, m):
    y = list(x)
    for i in range(D // 2):
        ang = m * BASE ** (-2.0 * i / D)
        a, b = x[i], x[i + D // 2]
        y[i] = a * math.cos(ang) - b * math.sin(ang)
        y[i + D // 2] = a * math.sin(ang) + b * math.cos(ang)
    return y


q, k, v = [], [], []
for t in range(2):
    a = rms(X[t], G_ATTN)
    q.append(rotate([s + b for s, b in zip(matvec(WQ, a), BQ)], POS[t]))
    k.append(rotate([s + b for s, b in zip(matvec(WK, a), BK)], POS[t]))
    v.append([s + b for s, b in zip(matvec(WV, a), BV)])

cache_k = [[0.0] * D for _ in range(8)]
cache_v = [[0.0] * D for _ in range(8)]
for t in range(2):  # the block's keys and values are written into the cache before the attention is taken
    cache_k[POS[t]], cache_v[POS[t]] = k[t], v[t]

out = []
for t in range(2):
    seen = range(POS[t] + 1)
    logits = [sum(q[t][c] * cache_k[j][c] for c in range(D)) / math.sqrt(D) for j in seen]
    mx = max(logits)
    w = [math.exp(s - mx) for s in logits]
    den = sum(w)
    o = [sum(w[j] / den * cache_v[j][c] for j in seen) for c in range(D)]
    x1 = [X[t][c] + y for c, y in enumerate(matvec(WO, o))]
    a2 = rms(x1, G_MLP)
    gate, up = matvec(WG, a2), matvec(WU, a2)
    h = [g / (1.0 + math.exp(-g)) * u for g, u in zip(gate, up)]
    out.append([x1[c] + y for c, y in enumerate(matvec(WD, h))])


def fmt(name, rows):
    return [name + " " + " ".join(repr(t) for t in row) for row in rows]


lines = ["# one decoder block, 2 tokens at positions 3 and 7 of an 8-slot cache (other slots zero), d=4, Hq=Hkv=1, D=4, F=3, base 100, eps 1e-5, half-split pairs",
         "# inputs: x g_attn g_mlp wq wk wv wo bq bk bv wg wu wd ; outputs: k v x_out (one row per token)"]
for name, rows in (("x", X), ("g_attn", [G_ATTN]), ("g_mlp", [G_MLP]), ("wq", WQ), ("wk", WK), ("wv", WV), ("wo", WO),
                   ("bq", [BQ]), ("bk", [BK]), ("bv", [BV]), ("wg", WG), ("wu", WU), ("wd", WD),
                   ("k", k), ("v", v), ("x_out", out)):
    lines += fmt(name, rows)
with open(os.path.join(os.path.dirname(__file__), "block_d4.txt"), "w") as f:
    f.write("\n".join(lines) + "\n")
