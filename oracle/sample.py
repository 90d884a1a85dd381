"""Plain CPU statement of sampling-mode verification (test infrastructure).

The approval of drafts compares, at every position, a token sampled from the model's conditional
distribution with the draft token ("Draft Construction and Verification"); the paper evaluates
temperature and top-p sampling (Figure 5) besides greedy choice.  The paper does not say how a
token is drawn.  The drawing rule stated here is exact integer arithmetic after one rounded
exponential per logit, so that two implementations that follow it agree bit for bit:

  1. m = max logit;  t_v = fl32(fl32(l_v - m) * c),  c = fl32(log2(e) / temperature)   (t_v <= 0)
  2. n = floor(t_v), f = t_v - n (exact);  r = P(f), the degree-6 polynomial below evaluated by
     Horner's rule in float32 with separately rounded multiplications and additions (1 <= r < 2,
     relative error against 2^f below 1e-7);  weight q_v = floor(r * 2^30) >> (-n)  (0 for n < -40):
     an unsigned fixed-point value of 2^t_v with 30 fractional bits; a logit of -inf has weight 0
  3. total = sum q_v;  need = ceil(total * floor(top_p * 65536) / 65536)
  4. nucleus = shortest prefix of the tokens ordered by (q descending, id ascending) whose weights
     sum to at least need;  Z = its sum
  5. target = floor(Z * floor(u * 2^24) / 2^24) for the uniform number u in [0, 1) supplied by the
     caller;  the sample is the first nucleus token IN ID ORDER whose running nucleus sum exceeds target.

Random numbers are inputs.  P(token = v) = q_v / Z on the nucleus up to 2^-24, i.e. the softmax of
logits / temperature restricted to the top-p nucleus and renormalised.
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np

# coefficients of P(f) ~ 2^f on [0, 1), lowest degree first (float32 values)
EXP2_COEF = [1.0, 0.6931470036506653, 0.24022991955280304, 0.0554824136197567, 0.009681269526481628,
             0.0012414311058819294, 0.00021795998327434063]
LOG2E = 1.4426950408889634


def weights(logits: Sequence[float], temperature: float) -> np.ndarray:
    """Steps 1-2: the fixed-point weight of every token (uint64 array)."""
    f32 = np.float32
    l = np.asarray(logits, dtype=f32)
    m = l.max()
    c = f32(f32(LOG2E) / f32(temperature))
    dead = np.isneginf(l)                      # a logit of -inf has weight 0
    t = ((np.where(dead, m, l) - m).astype(f32) * c).astype(f32)
    n = np.floor(t)
    f = (t - n).astype(f32)
    r = np.full_like(f, f32(EXP2_COEF[6]))
    for k in range(5, -1, -1):
        r = (r * f).astype(f32)
        r = (r + f32(EXP2_COEF[k])).astype(f32)
    big = np.floor(r.astype(np.float64) * 2.0 ** 30).astype(np.uint64)
    shift = (-n).astype(np.int64)
    q = np.where(shift <= 40, big >> np.minimum(shift, 40).astype(np.uint64), 0).astype(np.uint64)
    q[dead] = 0
    return q


def nucleus(q: np.ndarray, top_p: float) -> List[int]:
    """Steps 3-4: token ids of the nucleus (in the order they were taken)."""
    total = int(q.sum(dtype=np.uint64))
    p16 = int(np.floor(np.float64(np.float32(top_p)) * 65536.0))
    need = (total * p16 + 65535) >> 16
    order = sorted(range(len(q)), key=lambda v: (-int(q[v]), v))
    taken, s = [], 0
    for v in order:
        if s >= need:
            break
        taken.append(v)
        s += int(q[v])
    return taken


def sample(logits: Sequence[float], temperature: float, top_p: float, u: float) -> int:
    """One token drawn by the rule of the module header."""
    if not (temperature > 0.0 and 2.0 ** -16 <= top_p <= 1.0 and 0.0 <= u < 1.0):
        raise ValueError("temperature > 0, 2^-16 <= top_p <= 1, 0 <= u < 1")
    q = weights(logits, temperature)
    members = sorted(nucleus(q, top_p))
    z = sum(int(q[v]) for v in members)
    u24 = int(np.floor(np.float64(np.float32(u)) * 2.0 ** 24))
    target = (z * u24) >> 24
    run = 0
    for v in members:
        run += int(q[v])
        if run > target:
            return v
    raise AssertionError("unreachable: target < Z")


def chooser(temperature: float, top_p: float, u: Sequence[float]):
    """Per-node token choice for oracle.verify.verify(choose=...): node i draws with u[i] from its
    logits rounded to float32 (the precision the rule is stated in)."""
    def choose(logits: np.ndarray) -> np.ndarray:
        return sample_rows(np.asarray(logits, dtype=np.float32), temperature, top_p, u)
    return choose


def sample_rows(logits: np.ndarray, temperature: float, top_p: float, u: Sequence[float]) -> np.ndarray:
    return np.array([sample(logits[i], temperature, top_p, float(u[i])) for i in range(logits.shape[0])], dtype=np.int64)
