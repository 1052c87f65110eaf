"""Float64 CPU oracle of the per-layer MI hook.  TEST INFRASTRUCTURE ONLY.

This module is the slow, plain definition of what one hook call computes on a
ragged batch: every token row is dispatched by its slot id to a read primitive
(linear probe -> score), a write primitive (additive steering vector, or
ablation of a direction) or an SAE function (encode, activation, per-feature edits, decode, optional
reconstruction-error term); rows without an app are copied bit for bit.  It
follows the paper's description of the three primitives (Section 3,
"Read" / "Write" / "Conditional Write"), of the function contract (Section
4.2, "Executable units": activation slice + parameters in, derived signal
and/or activation update out), of buffers (Section 4.2, "State and dataflow")
and of inactive apps leaving a request untouched (Section 4.2, "Toggling
semantics").  The paper gives prose only; the formulas are the textbook ones
and the readings chosen where it is silent are listed in the design notes.

Only tests, the smoke entry and the benchmark's CPU-baseline leg may import
this module.  It shares no code with the CUDA path and imports nothing from
it.  All arithmetic is float64 on the exact bf16/fp32 input bits (bf16 ->
float64 is exact).  numpy's matmul and lexsort serve as library steps; there
is no blocking or reordering beyond converting weights in row chunks to bound
memory (each pre-activation is still one full-length dot product).

Parity pins: every function here is pinned by tests/test_oracle_pins.py
(closed forms, hand-worked values under tests/golden/, brute force, library
routines, algebraic invariants), tests/test_oracle_chain.py (slot chains) and
tests/test_oracle_fp8.py (8-bit encoder) and tests/test_oracle_fp8_act.py (8-bit encoder
input).  Nothing is "parity unpinned".
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, Iterable, List, Optional

import numpy as np

# kinds / enums restated here on purpose (the oracle depends on nothing else)
KIND_PROBE, KIND_STEER, KIND_SAE, KIND_PROJECT, KIND_ROUTER = 1, 2, 3, 4, 5
ACT_SIGMOID, ACT_SOFTMAX, ACT_NONE = 0, 1, 2
SAE_RELU, SAE_JUMPRELU, SAE_TOPK = 0, 1, 2
EDIT_CLAMP, EDIT_ABLATE = 0, 1
GATE_GE, GATE_LT = 0, 1

_CHUNK = 4096   # weight rows converted to float64 at a time


# ---------------------------------------------------------------------------
# bf16 <-> float64
# ---------------------------------------------------------------------------
def bf16_to_f64(bits) -> np.ndarray:
    """Exact value of bfloat16 bit patterns (uint16) as float64."""
    b = np.asarray(bits)
    if b.dtype != np.uint16:
        raise TypeError("bf16 data must be given as uint16 bit patterns, got %s" % b.dtype)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x) -> np.ndarray:
    """Round float64 to the nearest bfloat16 (ties to even); returns uint16 bits.
    bfloat16 = 1 sign, 8 exponent, 7 stored mantissa bits (8 significant)."""
    x = np.asarray(x, dtype=np.float64)
    sign = np.signbit(x)
    a = np.abs(x)
    m, e = np.frexp(a)                       # a = m * 2**e, m in [0.5, 1)
    # spacing of bf16 numbers around a: 2**(e-8) for normals, 2**-133 in the subnormal range
    qexp = np.maximum(e - 8, -133)
    q = np.ldexp(1.0, qexp)
    r = np.rint(a / q) * q                   # rint = round half to even; a/q is exact
    r = np.where(np.isfinite(a), r, a)
    with np.errstate(over="ignore"):          # beyond the largest bf16 the next line sets infinity
        r32 = r.astype(np.float32)           # exact: r has <= 8 significant bits
    r32 = np.where(r > 3.3895313892515355e38, np.float32(np.inf), r32)   # max bf16
    out = (r32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    out = np.where(np.isnan(x), np.uint16(0x7FC0), out)
    out = np.where(sign & ~np.isnan(x), out | np.uint16(0x8000), out)
    return out.astype(np.uint16)


# ---------------------------------------------------------------------------
# read primitive: linear probe  (Section 3, "Read")
# ---------------------------------------------------------------------------
def probe_scores(h: np.ndarray, W: np.ndarray, b: Optional[np.ndarray], act: int) -> np.ndarray:
    """h [d] float64, W [C, d] float64, b [C] or None -> scores [C].
    z_c = b_c + sum_i W[c,i] h[i]; sigmoid (C == 1), softmax, or the raw logit."""
    z = W @ h
    if b is not None:
        z = z + np.asarray(b, dtype=np.float64)
    if act == ACT_SIGMOID:
        return 1.0 / (1.0 + np.exp(-z))
    if act == ACT_SOFTMAX:
        e = np.exp(z - z.max())
        return e / e.sum()
    if act == ACT_NONE:
        return z
    raise ValueError("unknown probe activation %r" % act)


# ---------------------------------------------------------------------------
# write primitive: additive steering  (Section 3, "Write": add or subtract a vector)
# ---------------------------------------------------------------------------
def steer(h: np.ndarray, v: np.ndarray, alpha: float) -> np.ndarray:
    """h' = h + alpha * v   (alpha is an fp32 parameter, used at its exact value)."""
    return h + float(np.float32(alpha)) * v


def project(h: np.ndarray, r: np.ndarray, beta: float) -> np.ndarray:
    """Directional ablation, the usual statement of "subtract a vector" along a direction
    (Section 3, "Write"; Table 1, row 1):  h' = h - beta (h . r) r, with r used as given."""
    return h - float(np.float32(beta)) * float(h @ r) * r


# ---------------------------------------------------------------------------
# conditional write, activation-driven  (Section 3, "Conditional Write"; Section 4.1, the
# gate="probe(layer=18) >= 0" example; Section 4.2, "Activation and control semantics")
# ---------------------------------------------------------------------------
def gate_open(gate, t: int) -> bool:
    """The app applies to row t iff cmp(scores[t, column], threshold).  scores and threshold are
    fp32 values compared exactly; a NaN score fails either comparison."""
    v = float(np.float32(np.asarray(gate.scores)[t, gate.column]))
    thr = float(np.float32(gate.threshold))
    if gate.cmp == GATE_GE:
        return v >= thr
    if gate.cmp == GATE_LT:
        return v < thr
    raise ValueError("unknown gate comparison %r" % gate.cmp)


# ---------------------------------------------------------------------------
# SAE function
# ---------------------------------------------------------------------------
def _e4m3_value(c: np.ndarray) -> np.ndarray:
    c = np.asarray(c, dtype=np.int64)
    e, m = (c >> 3) & 0xF, c & 0x7
    mag = np.where(e == 0, (m / 8.0) * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64)))
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return np.where(c & 0x80, -mag, mag)


_E4M3_VALUES = _e4m3_value(np.arange(256))      # the definition, evaluated once for each of the 256 codes


def e4m3_to_f64(codes: np.ndarray) -> np.ndarray:
    """Value of 8-bit E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no
    infinities, S.1111.111 is NaN): +-2^(e-7) (1 + m/8) for e > 0, +-2^-6 (m/8) for e = 0."""
    return _E4M3_VALUES[np.asarray(codes, dtype=np.uint8)]


def encoder_rows_f64(W_enc_bits: np.ndarray, w_scale: Optional[np.ndarray] = None) -> np.ndarray:
    """Encoder rows as float64: bf16 bits, or (8-bit encoder) E4M3 codes times the row's fp32 scale."""
    if w_scale is None:
        return bf16_to_f64(W_enc_bits)
    return e4m3_to_f64(W_enc_bits) * np.asarray(w_scale, dtype=np.float64)[:, None]


E4M3_MAX = 448.0                                  # largest finite E4M3 magnitude (code 0x7E)
ACT_SCALE_MIN_EXP = -100                          # the row scale of the 8-bit input is never below 2^-100
_E4M3_GRID = _E4M3_VALUES[:127]                   # magnitudes of codes 0x00 .. 0x7E, ascending with the code


def e4m3_quantize(x: np.ndarray) -> np.ndarray:
    """Nearest E4M3 code of each entry of x (float64, |x| <= 448); a value half-way between two
    neighbouring codes goes to the even code (round-to-nearest-even of the 3-bit mantissa)."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    if np.any(a > E4M3_MAX):
        raise ValueError("e4m3_quantize takes magnitudes up to 448")
    hi = np.searchsorted(_E4M3_GRID, a, side="left")          # first code with value >= a
    hi = np.minimum(hi, 126)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - _E4M3_GRID[lo], _E4M3_GRID[hi] - a
    take_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(take_hi, hi, lo).astype(np.uint8)
    return np.where(np.signbit(x), code | 0x80, code).astype(np.uint8)


def act_row_scale(x: np.ndarray) -> float:
    """Scale of a row quantised to 8 bits: the smallest power of two s with max|x_i| / s <= 448,
    never below 2^-100; 1 for a row of zeros."""
    amax = float(np.max(np.abs(x))) if np.size(x) else 0.0
    if amax == 0.0:
        return 1.0
    m, E = math.frexp(amax)                          # amax = m 2^E, 0.5 <= m < 1;  448 = 0.875 * 2^9
    e = E - 9 if m <= 0.875 else E - 8
    return math.ldexp(1.0, max(e, ACT_SCALE_MIN_EXP))


def quantize_rows_e4m3(X: np.ndarray) -> np.ndarray:
    """What the 8-bit encoder sees in place of each row x of X: s * e4m3(code_i), with s = act_row_scale(x)
    and code_i the E4M3 code nearest to x_i / s."""
    X = np.atleast_2d(np.asarray(X, dtype=np.float64))
    out = np.empty_like(X)
    for n in range(X.shape[0]):
        s = act_row_scale(X[n])
        out[n] = e4m3_to_f64(e4m3_quantize(X[n] / s)) * s
    return out


def sae_preact(X: np.ndarray, W_enc_bits: np.ndarray, b_enc: np.ndarray,
               b_dec: Optional[np.ndarray] = None, center_input: bool = False,
               w_scale: Optional[np.ndarray] = None) -> np.ndarray:
    """Pre-activations z[n, j] = b_enc[j] + sum_i W_enc[j, i] * (X[n, i] - [center] b_dec[i]).
    X [n, d] float64; W_enc given as bf16 bits [S, d], or as E4M3 codes [S, d] with w_scale [S]."""
    X = np.atleast_2d(np.asarray(X, dtype=np.float64))
    if center_input and b_dec is not None:
        X = X - np.asarray(b_dec, dtype=np.float64)[None, :]
    S = W_enc_bits.shape[0]
    Z = np.empty((X.shape[0], S), dtype=np.float64)
    for j0 in range(0, S, _CHUNK):
        j1 = min(S, j0 + _CHUNK)
        Z[:, j0:j1] = X @ encoder_rows_f64(W_enc_bits[j0:j1], None if w_scale is None else w_scale[j0:j1]).T
    return Z + np.asarray(b_enc, dtype=np.float64)[None, :]


def topk_indices(z: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest entries of z, sorted by descending value; equal values
    are ordered (and therefore kept) by ascending index.  Brute force: a full sort."""
    idx = np.arange(z.shape[0])
    order = np.lexsort((idx, -z))            # primary key -z, secondary key idx
    return order[:k]


def sae_activate(z: np.ndarray, act: int, k: int = 0, theta: Optional[np.ndarray] = None,
                 K_override: Optional[np.ndarray] = None):
    """z [S] -> (f [S], K or None).
    ReLU: f = max(z, 0).  JumpReLU: f = z where z > theta (strict), else 0.
    TopK: K = the k largest PRE-activations; f_j = max(z_j, 0) for j in K, else 0."""
    if act == SAE_RELU:
        return np.maximum(z, 0.0), None
    if act == SAE_JUMPRELU:
        return np.where(z > np.asarray(theta, dtype=np.float64), z, 0.0), None
    if act == SAE_TOPK:
        K = topk_indices(z, k) if K_override is None else np.asarray(K_override, dtype=np.int64)
        f = np.zeros_like(z)
        f[K] = np.maximum(z[K], 0.0)
        return f, K
    raise ValueError("unknown SAE activation %r" % act)


def sae_edit(f: np.ndarray, idx, val, mode) -> np.ndarray:
    """Per-feature interventions on the post-activation vector: clamp SETS f_j = c
    (whether or not j was active), ablate sets f_j = 0.  Applied in list order."""
    g = f.copy()
    for j, c, m in zip(np.asarray(idx), np.asarray(val), np.asarray(mode)):
        if m == EDIT_CLAMP:
            g[int(j)] = float(np.float32(c))
        elif m == EDIT_ABLATE:
            g[int(j)] = 0.0
        else:
            raise ValueError("unknown edit mode %r" % m)
    return g


def sae_reconstruct(g: np.ndarray, W_dec_bits: np.ndarray, b_dec: Optional[np.ndarray]) -> np.ndarray:
    """xhat(g) = b_dec + sum_j g_j W_dec[j, :], summed over the nonzero g_j."""
    d = W_dec_bits.shape[1]
    out = np.zeros(d, dtype=np.float64) if b_dec is None else np.asarray(b_dec, dtype=np.float64).copy()
    nz = np.nonzero(g)[0]
    for c0 in range(0, len(nz), _CHUNK):
        jj = nz[c0:c0 + _CHUNK]
        out = out + g[jj] @ bf16_to_f64(W_dec_bits[jj])
    return out


def sae_row(x: np.ndarray, z: np.ndarray, sae, app, K_override=None):
    """One SAE row, literal form.  With the error term the output is
    xhat(f') + (x - xhat(f)), the error being taken from the UNEDITED features;
    without it the output is xhat(f').  Returns (y, K, n_active, f)."""
    f, K = sae_activate(z, sae.act, sae.k, sae.theta, K_override)
    f2 = sae_edit(f, app.edit_idx, app.edit_val, app.edit_mode)
    xhat_edit = sae_reconstruct(f2, sae.W_dec, sae.b_dec)
    if app.add_error:
        xhat = sae_reconstruct(f, sae.W_dec, sae.b_dec)
        y = xhat_edit + (x - xhat)
    else:
        y = xhat_edit
    return y, K, int(np.count_nonzero(f > 0.0)), f


def sae_row_delta(x: np.ndarray, z: np.ndarray, sae, app, K_override=None) -> np.ndarray:
    """The same row in delta form (error term on): x + sum over edited j of (f'_j - f_j) W_dec[j].
    A second, independent route to the same number; tests require it to agree with sae_row."""
    f, _ = sae_activate(z, sae.act, sae.k, sae.theta, K_override)
    f2 = sae_edit(f, app.edit_idx, app.edit_val, app.edit_mode)
    y = x.copy()
    for j in np.unique(np.asarray(app.edit_idx, dtype=np.int64)):
        y = y + (f2[j] - f[j]) * bf16_to_f64(sae.W_dec[int(j)])
    return y


# ---------------------------------------------------------------------------
# whole hook
# ---------------------------------------------------------------------------
@dataclass
class HookResult:
    rows: np.ndarray                        # token indices evaluated (ascending)
    y: Dict[int, np.ndarray] = field(default_factory=dict)        # row -> float64 [d] exact output
    out_bits: Dict[int, np.ndarray] = field(default_factory=dict)  # row -> uint16 [d] (bf16 of y; input bits if unmodified)
    modified: Dict[int, bool] = field(default_factory=dict)       # row -> hook wrote the row
    scores: Dict[int, np.ndarray] = field(default_factory=dict)   # probe rows only -> float64 [C]
    topk: Dict[int, np.ndarray] = field(default_factory=dict)     # TopK SAE rows -> K (descending z)
    z: Dict[int, np.ndarray] = field(default_factory=dict)        # SAE rows -> float64 [S] (if keep_z)
    n_active: Dict[int, int] = field(default_factory=dict)        # SAE rows
    kind: Dict[int, int] = field(default_factory=dict)            # row -> app kind, 0 = pass-through


def apply_hook(w, rows: Optional[Iterable[int]] = None, keep_z: bool = False,
               topk_override: Optional[Dict[int, np.ndarray]] = None) -> HookResult:
    """Evaluate the hook on a host workload (numpy arrays; bf16 as uint16 bits).

    for each row t:  s = token_slot[t] if t < T_live else -1
      s < 0, out of range, unregistered, or the slot's gate closed for row t
                                           -> pass-through (bits unchanged, no score)
      probe  -> scores[t, :C]; hidden unchanged
      steer  -> h + alpha v
      SAE    -> encode, activate, edit, decode (+ error term)
    `rows` restricts evaluation to a subset (rows are independent).  `topk_override`
    maps a row to a TopK index set to use instead of the oracle's own (for re-checking a
    row where a near-tie was legitimately resolved differently)."""
    T = w.T_max
    rows = np.arange(T) if rows is None else np.unique(np.asarray(list(rows), dtype=np.int64))
    res = HookResult(rows=rows)
    hidden_bits = w.hidden
    sae_rows: Dict[int, list] = {}
    for t in rows:
        t = int(t)
        s = int(w.token_slot[t]) if t < w.T_live else -1
        app = w.apps.get(s) if 0 <= s < w.n_slots_max else None
        if app is not None and app.kind == KIND_SAE and app.group not in w.groups:
            app = None
        if app is not None and getattr(app, "gate", None) is not None and not gate_open(app.gate, t):
            app = None                       # gate closed: the row passes through
        if app is None:
            res.kind[t] = 0
            res.modified[t] = False
            res.out_bits[t] = hidden_bits[t].copy()
            res.y[t] = bf16_to_f64(hidden_bits[t])
            continue
        res.kind[t] = app.kind
        h = bf16_to_f64(hidden_bits[t])
        if app.kind == KIND_PROBE:
            res.scores[t] = probe_scores(h, bf16_to_f64(app.W), app.b, app.act)
            res.modified[t] = False
            res.out_bits[t] = hidden_bits[t].copy()
            res.y[t] = h
        elif app.kind == KIND_STEER:
            y = steer(h, bf16_to_f64(app.v), app.alpha)
            res.modified[t] = True
            res.y[t] = y
            res.out_bits[t] = f64_to_bf16_bits(y)
        elif app.kind == KIND_PROJECT:
            y = project(h, bf16_to_f64(app.r), app.beta)
            res.modified[t] = True
            res.y[t] = y
            res.out_bits[t] = f64_to_bf16_bits(y)
        elif app.kind == KIND_ROUTER:            # acts on the router logits, not on the hidden state
            res.kind[t] = 0
            res.modified[t] = False
            res.out_bits[t] = hidden_bits[t].copy()
            res.y[t] = h
        elif app.kind == KIND_SAE:
            sae_rows.setdefault(app.group, []).append(t)
        else:
            raise ValueError("unknown app kind %r" % app.kind)
    for g, ts in sae_rows.items():
        sae = w.groups[g]
        X = bf16_to_f64(hidden_bits[np.asarray(ts)])
        X_enc = quantize_rows_e4m3(X) if getattr(w, "fp8_act", False) else X      # 8-bit input: the encode alone sees it
        Z = sae_preact(X_enc, sae.W_enc, sae.b_enc, sae.b_dec, sae.center_input, getattr(sae, "w_scale", None))
        for n, t in enumerate(ts):
            app = w.apps[int(w.token_slot[t])]
            Ko = None if topk_override is None else topk_override.get(t)
            y, K, n_act, _ = sae_row(X[n], Z[n], sae, app, Ko)
            res.modified[t] = True
            res.y[t] = y
            res.out_bits[t] = f64_to_bf16_bits(y)
            res.n_active[t] = n_act
            if K is not None:
                res.topk[t] = K
            if keep_z:
                res.z[t] = Z[n].copy()
    return res


# ---------------------------------------------------------------------------
# several apps on one row  (composition model: every app contributes its own hook functions and
# state and the runtime applies the active ones at the hook; "All Apps Combined" in the evaluation)
# ---------------------------------------------------------------------------
MAX_CHAIN = 4


def chain_slots(w, s: int) -> List[int]:
    """Slots applied, in order, to a row whose token slot is s: s, chains[s], chains[chains[s]], ...
    (at most MAX_CHAIN of them; the walk stops at a slot without a link or without an app)."""
    out: List[int] = []
    chains = getattr(w, "chains", None) or {}
    while 0 <= s < w.n_slots_max and s in w.apps and len(out) < MAX_CHAIN:
        out.append(s)
        if s not in chains:
            break
        s = int(chains[s])
    return out


@dataclass
class ChainResult:
    rows: np.ndarray
    out_bits: Dict[int, np.ndarray] = field(default_factory=dict)   # bf16 bits of the row after the last app
    y: Dict[int, np.ndarray] = field(default_factory=dict)          # float64 value the last write produced
    modified: Dict[int, bool] = field(default_factory=dict)
    scores: Dict[int, Dict[int, float]] = field(default_factory=dict)   # row -> {column: score}
    topk: Dict[int, np.ndarray] = field(default_factory=dict)
    n_active: Dict[int, int] = field(default_factory=dict)
    applied: Dict[int, List[int]] = field(default_factory=dict)     # slots whose app ran on the row


def apply_chain_hook(w, rows: Optional[Iterable[int]] = None,
                     topk_override: Optional[Dict[int, np.ndarray]] = None) -> ChainResult:
    """The hook with slot chains.  For row t the apps of chain_slots(w, token_slot[t]) are applied one
    after the other; each sees the row as the previous one left it, rounded to bf16 (exactly what
    separate hook calls on the bf16 residual stream would see).  Every app's gate is evaluated on its
    own: a closed gate skips that app only.  The probes of a chain write side by side: a probe's
    first column is the total class count of the chain's earlier probes (skipped ones included, so
    the layout does not depend on the data).  Router apps do not act on the hidden state."""
    T = w.T_max
    rows = np.arange(T) if rows is None else np.unique(np.asarray(list(rows), dtype=np.int64))
    res = ChainResult(rows=rows)
    for t in rows:
        t = int(t)
        s = int(w.token_slot[t]) if t < w.T_live else -1
        cur = w.hidden[t].copy()
        res.modified[t] = False
        res.scores[t] = {}
        res.applied[t] = []
        res.y[t] = bf16_to_f64(cur)
        col = 0
        for sl in chain_slots(w, s):
            app = w.apps[sl]
            n_cols = int(np.asarray(app.W).shape[0]) if app.kind == KIND_PROBE else 0
            first_col, col = col, col + n_cols
            if app.kind == KIND_SAE and app.group not in w.groups:
                continue
            if getattr(app, "gate", None) is not None and not gate_open(app.gate, t):
                continue
            h = bf16_to_f64(cur)
            if app.kind == KIND_PROBE:
                sc = probe_scores(h, bf16_to_f64(app.W), app.b, app.act)
                for c in range(n_cols):
                    res.scores[t][first_col + c] = float(sc[c])
            elif app.kind == KIND_STEER:
                y = steer(h, bf16_to_f64(app.v), app.alpha)
            elif app.kind == KIND_PROJECT:
                y = project(h, bf16_to_f64(app.r), app.beta)
            elif app.kind == KIND_SAE:
                sae = w.groups[app.group]
                h_enc = quantize_rows_e4m3(h[None, :]) if getattr(w, "fp8_act", False) else h[None, :]
                z = sae_preact(h_enc, sae.W_enc, sae.b_enc, sae.b_dec, sae.center_input,
                               getattr(sae, "w_scale", None))[0]
                Ko = None if topk_override is None else topk_override.get(t)
                y, K, n_act, _ = sae_row(h, z, sae, app, Ko)
                res.n_active[t] = n_act
                if K is not None:
                    res.topk[t] = K
            elif app.kind == KIND_ROUTER:
                continue
            else:
                raise ValueError("unknown app kind %r" % app.kind)
            res.applied[t].append(sl)
            if app.kind != KIND_PROBE:
                res.modified[t] = True
                res.y[t] = y
                cur = f64_to_bf16_bits(y)
        res.out_bits[t] = cur
    return res


# ---------------------------------------------------------------------------
# router-logit steering  (Table 1, row 7: a conditional write on the MoE router logits)
# ---------------------------------------------------------------------------
def apply_router_hook(w, logits: np.ndarray) -> np.ndarray:
    """logits fp32 [T, E] -> float64 [T, E]: rows whose slot holds a router app with E experts (and
    an open gate) get logits + delta; every other row is returned unchanged."""
    out = np.asarray(logits, dtype=np.float64).copy()
    E = out.shape[1]
    for t in range(min(w.T_live, w.T_max)):
        s = int(w.token_slot[t])
        app = w.apps.get(s) if 0 <= s < w.n_slots_max else None
        if app is None or app.kind != KIND_ROUTER or len(app.delta) != E:
            continue
        if getattr(app, "gate", None) is not None and not gate_open(app.gate, t):
            continue
        out[t] = out[t] + np.asarray(app.delta, dtype=np.float64)
    return out
