"""Plain data containers for one MI-hook workload.

A workload is everything one hook call sees: the hidden states of a ragged
batch, the token->slot map, and the registered MI functions (probes, steering
vectors, SAE weight sets and the per-slot SAE edit lists).  This module holds
data only: none of the hook's arithmetic lives here, so both the CPU oracle
and the CUDA path can be fed from it without sharing any of the method.

Tensors are torch tensors on whatever device the generator was asked for;
`host()` turns a workload into numpy arrays (bf16 tensors become their raw
uint16 bit patterns, so the oracle sees exactly the bits the GPU sees).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np
import torch

# app kinds
KIND_PROBE, KIND_STEER, KIND_SAE, KIND_PROJECT, KIND_ROUTER = 1, 2, 3, 4, 5
# probe activations
ACT_SIGMOID, ACT_SOFTMAX, ACT_NONE = 0, 1, 2
# SAE activations
SAE_RELU, SAE_JUMPRELU, SAE_TOPK = 0, 1, 2
# edit modes
EDIT_CLAMP, EDIT_ABLATE = 0, 1


GATE_GE, GATE_LT = 0, 1


@dataclass
class Gate:
    """Activation-driven condition: the app applies to row t iff cmp(scores[t, column], threshold)."""
    scores: object            # fp32 [T_max, stride]
    column: int
    cmp: int                  # GATE_GE | GATE_LT
    threshold: float


@dataclass
class Probe:
    W: object                 # bf16 [C, d] (torch) or uint16 bits (numpy)
    b: object                 # fp32 [C]
    act: int
    kind: int = KIND_PROBE
    gate: Optional[Gate] = None

    @property
    def n_classes(self) -> int:
        return int(self.W.shape[0])


@dataclass
class Steer:
    v: object                 # bf16 [d]
    alpha: float
    kind: int = KIND_STEER
    gate: Optional[Gate] = None


@dataclass
class Project:
    r: object                 # bf16 [d], used as given
    beta: float
    kind: int = KIND_PROJECT
    gate: Optional[Gate] = None


@dataclass
class Router:
    delta: object             # fp32 [n_experts], added to the router logits
    kind: int = KIND_ROUTER
    gate: Optional[Gate] = None


@dataclass
class SaeWeights:
    d_sae: int
    act: int
    k: int                    # TopK only (0 otherwise)
    W_enc: object             # bf16 [d_sae, d]; row j = encoder direction j.  With w_scale set: uint8 [d_sae, d], E4M3 codes
    b_enc: object             # fp32 [d_sae]
    W_dec: object             # bf16 [d_sae, d]; row j = decoder direction j
    theta: Optional[object] = None   # fp32 [d_sae], JumpReLU only
    b_dec: Optional[object] = None   # fp32 [d]
    center_input: bool = False
    w_scale: Optional[object] = None   # fp32 [d_sae]: 8-bit encoder, W_enc[j, i] = e4m3(code[j, i]) * w_scale[j]


@dataclass
class SaeApp:
    group: int
    edit_idx: np.ndarray      # int32 [r]
    edit_val: np.ndarray      # fp32 [r]   (clamp target; ignored for ablate)
    edit_mode: np.ndarray     # uint8 [r]  EDIT_CLAMP | EDIT_ABLATE
    add_error: bool
    kind: int = KIND_SAE
    gate: Optional[Gate] = None


@dataclass
class Workload:
    name: str
    d_model: int
    T_max: int
    T_live: int
    hidden: object                      # bf16 [T_max, d]
    token_slot: np.ndarray              # int32 [T_max], -1 = no app
    apps: Dict[int, object] = field(default_factory=dict)
    groups: Dict[int, SaeWeights] = field(default_factory=dict)
    n_slots_max: int = 0
    n_groups_max: int = 0
    C_max: int = 1
    k_max: int = 0
    r_max: int = 0
    d_sae_max: int = 0
    meta: dict = field(default_factory=dict)
    chains: Dict[int, int] = field(default_factory=dict)   # slot -> next slot applied to the same row
    fp8_act: bool = False               # SAE rows reach the (8-bit) encoder quantised to E4M3 with a power-of-two row scale


def bits(t):
    """bf16 torch tensor -> numpy uint16 bit patterns (host)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t
    if t.dtype == torch.bfloat16:
        return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
    return t.detach().cpu().contiguous().numpy()


def from_bits(a: np.ndarray, device="cpu"):
    """numpy uint16 bit patterns -> bf16 torch tensor."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


def host(w: Workload, only_groups=None) -> Workload:
    """Copy of the workload with every tensor as a numpy array (bf16 -> uint16 bits).
    `only_groups` keeps just those SAE weight sets (large configs: copying 32 GiB of weights to
    the host to check a few rows is pointless); apps of the other sets then count as unhooked."""
    apps = {}
    for s, a in w.apps.items():
        g = None if a.gate is None else Gate(bits(a.gate.scores), a.gate.column, a.gate.cmp, a.gate.threshold)
        if a.kind == KIND_PROBE:
            apps[s] = Probe(bits(a.W), bits(a.b), a.act, gate=g)
        elif a.kind == KIND_STEER:
            apps[s] = Steer(bits(a.v), float(a.alpha), gate=g)
        elif a.kind == KIND_PROJECT:
            apps[s] = Project(bits(a.r), float(a.beta), gate=g)
        elif a.kind == KIND_ROUTER:
            apps[s] = Router(bits(a.delta), gate=g)
        else:
            apps[s] = SaeApp(a.group, a.edit_idx, a.edit_val, a.edit_mode, a.add_error, gate=g)
    groups = {
        g: SaeWeights(sw.d_sae, sw.act, sw.k, bits(sw.W_enc), bits(sw.b_enc), bits(sw.W_dec),
                      bits(sw.theta), bits(sw.b_dec), sw.center_input, bits(sw.w_scale))
        for g, sw in w.groups.items() if only_groups is None or g in only_groups
    }
    return Workload(w.name, w.d_model, w.T_max, w.T_live, bits(w.hidden), w.token_slot.copy(),
                    apps, groups, w.n_slots_max, w.n_groups_max, w.C_max, w.k_max, w.r_max,
                    w.d_sae_max, dict(w.meta), dict(w.chains), w.fp8_act)
