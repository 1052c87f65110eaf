"""Register a workload's apps with a hook context (any object with the binding's method names)."""
from __future__ import annotations

from .spec import KIND_PROBE, KIND_PROJECT, KIND_ROUTER, KIND_SAE, KIND_STEER, Workload


def make_context(mix_cls, w: Workload, flags: int = 0, **over):
    """Create a context sized for workload `w` and register everything in it."""
    kw = dict(d_model=w.d_model, T_max=w.T_max, n_slots_max=max(w.n_slots_max, 1), n_groups_max=w.n_groups_max,
              C_max=max(w.C_max, 1), k_max=w.k_max, r_max=w.r_max, d_sae_max=w.d_sae_max, flags=flags)
    kw.update(over)
    m = mix_cls(**kw)
    install(m, w)
    return m


def install(m, w: Workload):
    for g, sw in w.groups.items():
        m.register_sae_weights(g, sw.d_sae, sw.act, sw.k, sw.W_enc, sw.b_enc, sw.W_dec, theta=sw.theta,
                               b_dec=sw.b_dec, center_input=sw.center_input, w_scale=getattr(sw, "w_scale", None))
    for s, a in w.apps.items():
        if a.kind == KIND_PROBE:
            m.register_probe(s, a.W, a.b, a.act)
        elif a.kind == KIND_STEER:
            m.register_steer(s, a.v, a.alpha)
        elif a.kind == KIND_PROJECT:
            m.register_project(s, a.r, a.beta)
        elif a.kind == KIND_ROUTER:
            m.register_router(s, a.delta)
        elif a.kind == KIND_SAE:
            m.register_sae_app(s, a.group, a.edit_idx, a.edit_val, a.edit_mode, a.add_error)
        if getattr(a, "gate", None) is not None:
            m.set_gate(s, a.gate.scores, a.gate.column, a.gate.cmp, a.gate.threshold)
    for s, nxt in getattr(w, "chains", {}).items():
        m.set_chain(s, nxt)
    m.set_slot_map(w.token_slot, w.T_live)
