"""Seeded synthetic workloads shaped like the five benchmark configurations.

Everything here is input generation: random tensors with the stated
distributions, ragged request lengths, and the assignment of requests to app
slots.  No step of the hook itself is computed here.

Real-valued tensors come from a `torch.Generator` on the requested device
(fp32 draw -> transform -> round to bf16); integer structure (lengths, slot
assignment, edit lists) comes from `numpy.random.default_rng`.  The CPU and
CUDA generators give different streams, so a parity test generates once and
hands the SAME bits to both sides (`spec.host`).

Seeds: config c uses BASE_SEED + 1000*c; replay r of config 4 uses
BASE_SEED + 4000 + r.
"""
from __future__ import annotations

from typing import Callable, Optional

import numpy as np
import torch

from .spec import (ACT_SIGMOID, ACT_SOFTMAX, EDIT_ABLATE, EDIT_CLAMP, SAE_JUMPRELU, SAE_TOPK,
                   ACT_NONE, Probe, Project, SaeApp, SaeWeights, Steer, Workload)

BASE_SEED = 20260722

CONFIG_NAMES = ["tiny", "decode", "sae_heavy", "mixed", "replay"]

# An edit hint maps (group id, SaeWeights, bf16 hidden row [d]) -> indices of
# features that are active on that row.  It lets half of a request's edits
# land on features that actually fire (a uniformly random feature of a
# 65536-wide TopK-64 SAE is active 0.1 % of the time).  The caller supplies it
# (tests pass the oracle's encoder); without one every index is uniform.
EditHint = Callable[[int, SaeWeights, torch.Tensor], np.ndarray]


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn_bf16(g, device, rows, cols, std, chunk_rows=16384):
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device=device)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        x = torch.randn((r1 - r0, cols), generator=g, device=device, dtype=torch.float32)
        out[r0:r1] = (x * std).to(torch.bfloat16)
    return out


def _unit_rows_bf16(g, device, rows, cols, chunk_rows=16384):
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device=device)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        x = torch.randn((r1 - r0, cols), generator=g, device=device, dtype=torch.float32)
        x = x / x.norm(dim=1, keepdim=True)
        out[r0:r1] = x.to(torch.bfloat16)
    return out


def _hidden(g, device, T, d, outlier_cols=None):
    x = torch.randn((T, d), generator=g, device=device, dtype=torch.float32)
    if outlier_cols is not None and len(outlier_cols):
        x[:, torch.as_tensor(outlier_cols, device=device, dtype=torch.long)] *= 20.0
    return x.to(torch.bfloat16)


def make_sae_weights(g, device, d, d_sae, act, k=0, theta_range=None, b_enc_mean=-0.1, fp8=False):
    """W_enc ~ N(0, 1/d) (variance), W_dec rows unit-norm, b_enc ~ N(mean, std 0.02).
    fp8: the encoder is stored as E4M3 codes with one fp32 scale per feature (row absmax / 448),
    rounded by torch's float8_e4m3fn conversion; the codes and scales ARE the weights."""
    w_scale = None
    if fp8:
        Wf = torch.randn((d_sae, d), generator=g, device=device, dtype=torch.float32) * d ** -0.5
        w_scale = (Wf.abs().amax(dim=1) / 448.0).clamp_min(1e-12)
        W_enc = (Wf / w_scale[:, None]).to(torch.float8_e4m3fn).view(torch.uint8)
    else:
        W_enc = _randn_bf16(g, device, d_sae, d, d ** -0.5)
    W_dec = _unit_rows_bf16(g, device, d_sae, d)
    b_enc = (torch.randn((d_sae,), generator=g, device=device, dtype=torch.float32) * 0.02 + b_enc_mean)
    theta = None
    if act == SAE_JUMPRELU:
        lo, hi = theta_range
        theta = torch.rand((d_sae,), generator=g, device=device, dtype=torch.float32) * (hi - lo) + lo
    return SaeWeights(d_sae=d_sae, act=act, k=k, W_enc=W_enc, b_enc=b_enc, W_dec=W_dec, theta=theta, w_scale=w_scale)


def ragged_lengths_uniform(rng, T, R):
    """R positive lengths summing to T: 1 + multinomial(T - R, uniform)."""
    assert T >= R
    return (1 + rng.multinomial(T - R, np.full(R, 1.0 / R))).astype(np.int64)


def ragged_lengths_lognormal(rng, T, R, mu=5.0, sigma=1.0, cap=2048):
    """R lengths ~ lognormal(mu, sigma) capped at `cap`, rescaled to sum to T."""
    cap = min(cap, T)
    raw = np.clip(np.rint(rng.lognormal(mu, sigma, size=R)), 1, cap)
    lens = raw.copy()
    for _ in range(64):
        s = lens.sum()
        if s == T:
            break
        lens = np.clip(np.rint(lens * (T / s)), 1, cap)
        diff = int(T - lens.sum())
        order = np.argsort(-lens, kind="stable")
        i = 0
        while diff != 0 and i < 16 * R:
            j = order[i % R]
            step = 1 if diff > 0 else -1
            if 1 <= lens[j] + step <= cap:
                lens[j] += step
                diff -= step
            i += 1
    assert lens.sum() == T, (lens.sum(), T)
    return lens.astype(np.int64)


def _token_slot_from_requests(lengths, req_slot, order, T_max):
    """Requests occupy contiguous token ranges, laid out in `order`."""
    token_slot = np.full(T_max, -1, dtype=np.int32)
    token_req = np.full(T_max, -1, dtype=np.int32)
    t = 0
    for r in order:
        n = int(lengths[r])
        token_slot[t:t + n] = req_slot[r]
        token_req[t:t + n] = r
        t += n
    return token_slot, token_req, t


def _edits(rng, d_sae, n_edit, active: Optional[np.ndarray]):
    """n_edit distinct feature ids: half from `active` (if given), half uniform.
    First half of the list clamps to U[2, 8], second half ablates."""
    chosen = []
    if active is not None and len(active):
        take = min(n_edit // 2, len(active))
        chosen = list(rng.choice(np.asarray(active), size=take, replace=False))
    while len(chosen) < n_edit:
        j = int(rng.integers(0, d_sae))
        if j not in chosen:
            chosen.append(j)
    idx = np.asarray(chosen, dtype=np.int32)
    rng.shuffle(idx)
    mode = np.where(np.arange(n_edit) < n_edit // 2, EDIT_CLAMP, EDIT_ABLATE).astype(np.uint8)
    val = np.where(mode == EDIT_CLAMP, rng.uniform(2.0, 8.0, size=n_edit), 0.0).astype(np.float32)
    return idx, val, mode


def _last_row_of_request(token_req, r):
    rows = np.nonzero(token_req == r)[0]
    return int(rows[-1]) if len(rows) else -1


# --------------------------------------------------------------------------
# config 0: tiny
# --------------------------------------------------------------------------
def make_tiny(device="cpu", d=512, T=64, d_sae=4096, k=32, seed=None):
    seed = BASE_SEED if seed is None else seed
    g, rng = _gen(device, seed), np.random.default_rng(seed)
    R = 8
    hidden = _hidden(g, device, T, d)
    lengths = ragged_lengths_uniform(rng, T, R)
    probe = Probe(W=_randn_bf16(g, device, 1, d, d ** -0.5),
                  b=torch.zeros(1, dtype=torch.float32, device=device), act=ACT_SIGMOID)
    steer = Steer(v=_unit_rows_bf16(g, device, 1, d)[0].contiguous(), alpha=4.0)
    sae = make_sae_weights(g, device, d, d_sae, SAE_TOPK, k=k)
    cidx = rng.choice(d_sae, size=4, replace=False).astype(np.int32)
    cval = np.full(4, 5.0, dtype=np.float32)
    cmode = np.full(4, EDIT_CLAMP, dtype=np.uint8)
    apps = {0: probe, 1: steer,
            2: SaeApp(0, cidx, cval, cmode, add_error=True),
            3: SaeApp(0, cidx.copy(), cval.copy(), cmode.copy(), add_error=False)}
    req_slot = np.array([0, 0, 1, 1, 2, 3, -1, -1], dtype=np.int32)
    rng.shuffle(req_slot)
    order = rng.permutation(R)
    token_slot, token_req, used = _token_slot_from_requests(lengths, req_slot, order, T)
    assert used == T
    return Workload("tiny", d, T, T, hidden, token_slot, apps, {0: sae}, n_slots_max=8,
                    n_groups_max=1, C_max=1, k_max=k, r_max=4, d_sae_max=d_sae,
                    meta={"lengths": lengths, "req_slot": req_slot, "token_req": token_req, "seed": seed})


# --------------------------------------------------------------------------
# several apps on one row ("all apps combined"): slot chains
# --------------------------------------------------------------------------
def make_chained(device="cpu", d=512, T=300, d_sae=2048, k=16, C=5, seed=None):
    """Every hooked request carries a chain of apps on each of its tokens:
         0 -> 1 -> 2 -> 3   sigmoid probe, steering, softmax probe (C classes), TopK SAE edit (error term on)
         4 -> 5             projection, JumpReLU SAE edit (error term off)
         6 -> 1 -> ...      a second head that joins the first chain at its steering app
         7                  a steering app on its own; 8: a raw-logit probe on its own
       plus requests that enter chain 0 in the middle (token slot 1, 2 or 3) and unhooked requests."""
    seed = BASE_SEED + 5000 if seed is None else seed
    g, rng = _gen(device, seed), np.random.default_rng(seed)
    hidden = _hidden(g, device, T, d)
    zero1 = torch.zeros(1, dtype=torch.float32, device=device)
    sae_t = make_sae_weights(g, device, d, d_sae, SAE_TOPK, k=k)
    sae_j = make_sae_weights(g, device, d, d_sae, SAE_JUMPRELU, k=0, theta_range=(0.05, 0.3), b_enc_mean=-2.0)
    e_t = rng.choice(d_sae, size=4, replace=False).astype(np.int32)
    e_j = rng.choice(d_sae, size=3, replace=False).astype(np.int32)
    apps = {
        0: Probe(W=_randn_bf16(g, device, 1, d, d ** -0.5), b=zero1.clone(), act=ACT_SIGMOID),
        1: Steer(v=_unit_rows_bf16(g, device, 1, d)[0].contiguous(), alpha=4.0),
        2: Probe(W=_randn_bf16(g, device, C, d, d ** -0.5),
                 b=torch.randn(C, generator=g, device=device, dtype=torch.float32), act=ACT_SOFTMAX),
        3: SaeApp(0, e_t, np.array([5.0, 0.0, 2.5, 0.0], np.float32),
                  np.array([EDIT_CLAMP, EDIT_ABLATE, EDIT_CLAMP, EDIT_ABLATE], np.uint8), add_error=True),
        4: Project(r=_unit_rows_bf16(g, device, 1, d)[0].contiguous(), beta=1.0),
        5: SaeApp(1, e_j, np.array([3.0, 0.0, 1.0], np.float32),
                  np.array([EDIT_CLAMP, EDIT_ABLATE, EDIT_CLAMP], np.uint8), add_error=False),
        6: Probe(W=_randn_bf16(g, device, 1, d, d ** -0.5), b=None, act=ACT_SIGMOID),
        7: Steer(v=_unit_rows_bf16(g, device, 1, d)[0].contiguous(), alpha=-2.0),
        8: Probe(W=_randn_bf16(g, device, 1, d, d ** -0.5), b=zero1.clone(), act=ACT_NONE),
    }
    chains = {0: 1, 1: 2, 2: 3, 4: 5, 6: 1}
    R = max(T // 12, 10)
    lengths = ragged_lengths_uniform(rng, T, R)
    req_slot = rng.choice(np.array([0, 0, 0, 4, 4, 6, 6, 7, 8, 1, 2, 3, 5, -1, -1], dtype=np.int32), size=R)
    req_slot[:10] = np.array([0, 4, 6, 7, 8, 1, 2, 3, 5, -1], dtype=np.int32)     # every case at least once
    rng.shuffle(req_slot)
    order = rng.permutation(R)
    token_slot, token_req, used = _token_slot_from_requests(lengths, req_slot, order, T)
    return Workload("chained", d, T, used, hidden, token_slot, apps, {0: sae_t, 1: sae_j}, n_slots_max=9,
                    n_groups_max=2, C_max=1 + C + 1, k_max=k, r_max=4, d_sae_max=d_sae,
                    meta={"lengths": lengths, "req_slot": req_slot, "token_req": token_req, "seed": seed},
                    chains=chains)


# --------------------------------------------------------------------------
# config 1: decode step
# --------------------------------------------------------------------------
def make_decode(device="cpu", d=4096, T=256, n_probe=64, n_steer=32, seed=None):
    seed = BASE_SEED + 1000 if seed is None else seed
    g, rng = _gen(device, seed), np.random.default_rng(seed)
    n_out = int(np.floor(0.001 * d))
    outliers = rng.choice(d, size=n_out, replace=False) if n_out else np.zeros(0, dtype=np.int64)
    hidden = _hidden(g, device, T, d, outliers)
    apps = {}
    Wp = _randn_bf16(g, device, n_probe, d, d ** -0.5)
    for i in range(n_probe):
        apps[i] = Probe(W=Wp[i:i + 1].contiguous(), b=torch.zeros(1, dtype=torch.float32, device=device),
                        act=ACT_SIGMOID)
    Vs = _unit_rows_bf16(g, device, n_steer, d)
    alphas = rng.uniform(1.0, 8.0, size=n_steer)
    for i in range(n_steer):
        apps[n_probe + i] = Steer(v=Vs[i].contiguous(), alpha=float(np.float32(alphas[i])))
    n_apps = n_probe + n_steer
    n_unhooked = T // 4
    req_slot = np.full(T, -1, dtype=np.int32)
    req_slot[n_unhooked:] = np.arange(T - n_unhooked) % n_apps
    rng.shuffle(req_slot)
    token_slot = req_slot.copy()           # one token per request
    return Workload("decode", d, T, T, hidden, token_slot, apps, {}, n_slots_max=n_apps,
                    n_groups_max=0, C_max=1, k_max=0, r_max=0, d_sae_max=0,
                    meta={"outlier_cols": outliers, "seed": seed})


# --------------------------------------------------------------------------
# config 2: SAE-heavy
# --------------------------------------------------------------------------
def make_sae_heavy(device="cpu", d=4096, d_sae=65536, k=64, T=512, R=32, G=4, n_edit=16,
                   edit_hint: Optional[EditHint] = None, seed=None, fp8=False, fp8_act=False):
    seed = BASE_SEED + 2000 if seed is None else seed
    g, rng = _gen(device, seed), np.random.default_rng(seed)
    hidden = _hidden(g, device, T, d)
    lengths = ragged_lengths_uniform(rng, T, R)
    groups = {gi: make_sae_weights(g, device, d, d_sae, SAE_TOPK, k=k, fp8=fp8) for gi in range(G)}
    req_slot = np.arange(R, dtype=np.int32)          # one app slot per request
    req_group = np.arange(R) % G
    order = rng.permutation(R)
    token_slot, token_req, used = _token_slot_from_requests(lengths, req_slot, order, T)
    apps = {}
    for r in range(R):
        gi = int(req_group[r])
        active = None
        if edit_hint is not None:
            active = edit_hint(gi, groups[gi], hidden[_last_row_of_request(token_req, r)])
        idx, val, mode = _edits(rng, d_sae, n_edit, active)
        apps[r] = SaeApp(gi, idx, val, mode, add_error=True)
    return Workload("sae_heavy", d, T, T, hidden, token_slot, apps, groups, n_slots_max=R,
                    n_groups_max=G, C_max=1, k_max=k, r_max=n_edit, d_sae_max=d_sae,
                    meta={"lengths": lengths, "token_req": token_req, "req_group": req_group, "seed": seed},
                    fp8_act=bool(fp8_act))


# --------------------------------------------------------------------------
# config 3: mixed chunked prefill + decode
# --------------------------------------------------------------------------
def make_mixed(device="cpu", d=5120, T=8192, R=64, d_sae=32768, C=16, n_probe=8, n_steer=8, G=2,
               n_edit=16, cap=2048, mu=5.0, b_enc_mean=-0.1,
               edit_hint: Optional[EditHint] = None, seed=None, fp8=False, fp8_act=False):
    seed = BASE_SEED + 3000 if seed is None else seed
    g, rng = _gen(device, seed), np.random.default_rng(seed)
    hidden = _hidden(g, device, T, d)
    lengths = ragged_lengths_lognormal(rng, T, R, mu=mu, cap=cap)
    apps = {}
    for i in range(n_probe):
        apps[i] = Probe(W=_randn_bf16(g, device, C, d, d ** -0.5),
                        b=torch.zeros(C, dtype=torch.float32, device=device), act=ACT_SOFTMAX)
    Vs = _unit_rows_bf16(g, device, n_steer, d)
    alphas = rng.uniform(1.0, 8.0, size=n_steer)
    for i in range(n_steer):
        apps[n_probe + i] = Steer(v=Vs[i].contiguous(), alpha=float(np.float32(alphas[i])))
    groups = {gi: make_sae_weights(g, device, d, d_sae, SAE_JUMPRELU, theta_range=(0.05, 0.3),
                                   b_enc_mean=b_enc_mean, fp8=fp8) for gi in range(G)}
    # deal requests (in a seeded order) unhooked until >= 30 % of rows, rest round-robin
    deal = rng.permutation(R)
    req_kind = np.zeros(R, dtype=np.int64)           # 0 none, 1 probe, 2 steer, 3 sae
    rows_unhooked, i = 0, 0
    while rows_unhooked < 0.30 * T and i < R:
        req_kind[deal[i]] = 0
        rows_unhooked += lengths[deal[i]]
        i += 1
    rr = 0
    for r in deal[i:]:
        req_kind[r] = 1 + rr % 3
        rr += 1
    req_slot = np.full(R, -1, dtype=np.int32)
    base_sae = n_probe + n_steer
    n_p = n_s = n_a = 0
    req_group = np.full(R, -1)
    for r in range(R):
        if req_kind[r] == 1:
            req_slot[r] = n_p % n_probe; n_p += 1
        elif req_kind[r] == 2:
            req_slot[r] = n_probe + n_s % n_steer; n_s += 1
        elif req_kind[r] == 3:
            req_slot[r] = base_sae + n_a; req_group[r] = n_a % G; n_a += 1
    order = rng.permutation(R)
    token_slot, token_req, used = _token_slot_from_requests(lengths, req_slot, order, T)
    for r in range(R):
        if req_kind[r] == 3:
            gi = int(req_group[r])
            active = None
            if edit_hint is not None:
                active = edit_hint(gi, groups[gi], hidden[_last_row_of_request(token_req, r)])
            idx, val, mode = _edits(rng, d_sae, n_edit, active)
            apps[int(req_slot[r])] = SaeApp(gi, idx, val, mode, add_error=True)
    return Workload("mixed", d, T, T, hidden, token_slot, apps, groups,
                    n_slots_max=base_sae + max(n_a, 1), n_groups_max=G, C_max=C, k_max=0,
                    r_max=n_edit, d_sae_max=d_sae,
                    meta={"lengths": lengths, "token_req": token_req, "req_kind": req_kind,
                          "req_group": req_group, "seed": seed}, fp8_act=bool(fp8_act))


# --------------------------------------------------------------------------
# config 4: fixed-size graph replay
# --------------------------------------------------------------------------
def make_replay(device="cpu", d=8192, T_max=2048, d_sae=131072, k=128, G=8, n_probe=64, n_steer=16,
                n_sae_slots=64, n_edit=16, seed=None, fp8=False, fp8_act=False):
    """Apps for the replay config; the slot map of each replay comes from `replay_map`."""
    seed = BASE_SEED + 4000 if seed is None else seed
    g, rng = _gen(device, seed), np.random.default_rng(seed)
    hidden = _hidden(g, device, T_max, d)
    apps = {}
    Wp = _randn_bf16(g, device, n_probe, d, d ** -0.5)
    for i in range(n_probe):
        apps[i] = Probe(W=Wp[i:i + 1].contiguous(), b=torch.zeros(1, dtype=torch.float32, device=device),
                        act=ACT_SIGMOID)
    Vs = _unit_rows_bf16(g, device, n_steer, d)
    alphas = rng.uniform(1.0, 8.0, size=n_steer)
    for i in range(n_steer):
        apps[n_probe + i] = Steer(v=Vs[i].contiguous(), alpha=float(np.float32(alphas[i])))
    groups = {gi: make_sae_weights(g, device, d, d_sae, SAE_TOPK, k=k, fp8=fp8) for gi in range(G)}
    base = n_probe + n_steer
    for i in range(n_sae_slots):
        idx, val, mode = _edits(rng, d_sae, n_edit, None)
        apps[base + i] = SaeApp(i % G, idx, val, mode, add_error=True)
    token_slot = np.full(T_max, -1, dtype=np.int32)
    w = Workload("replay", d, T_max, 0, hidden, token_slot, apps, groups,
                 n_slots_max=base + n_sae_slots, n_groups_max=G, C_max=1, k_max=k, r_max=n_edit,
                 d_sae_max=d_sae, meta={"seed": seed}, fp8_act=bool(fp8_act))
    return w


def replay_map(w: Workload, r: int):
    """Slot map of replay r: live rows are a prefix of n_live ~ U{0..T_max} rows (replays 0
    and 1 forced to 0 and T_max), cut into request segments of length 1 (prob 1/2) or
    U{2..256}; each segment is unhooked with prob 0.2, else a uniformly drawn slot."""
    rng = np.random.default_rng(w.meta["seed"] + r)
    T_max = w.T_max
    n_live = int(rng.integers(0, T_max + 1))
    if r == 0:
        n_live = 0
    elif r == 1:
        n_live = T_max
    slots = np.array(sorted(w.apps.keys()), dtype=np.int32)
    token_slot = np.full(T_max, -1, dtype=np.int32)
    t = 0
    while t < n_live:
        seg = 1 if rng.random() < 0.5 else int(rng.integers(2, 257))
        seg = min(seg, n_live - t)
        s = -1 if rng.random() < 0.2 else int(slots[rng.integers(0, len(slots))])
        token_slot[t:t + seg] = s
        t += seg
    return token_slot, n_live


def make_config(idx: int, device="cpu", **kw) -> Workload:
    return [make_tiny, make_decode, make_sae_heavy, make_mixed, make_replay][idx](device=device, **kw)
