// Slot -> app lookup shared by the kernels that read the slot map: the 48-byte app entry in three
// 16-byte loads, the slot's gate, and the status bit for bad slot ids.
#pragma once

#include "mix_internal.h"

namespace mix {

struct RowApp {
  bool gated;           // the slot has a gate (whether or not it let this row through)
  bool chained;         // another app follows on the same row (set even when the gate is closed)
  int raw_kind;         // the slot's kind even when the gate is closed (0: no valid app)
  int kind, C, act;     // kind 0: nothing to do
  float alpha;
  const uint4* W;
  const float* b;
};

// Does row t pass the gate of its slot?  (NaN fails both comparisons.)
__device__ __forceinline__ bool gate_open(const GateEntry* __restrict__ gates, int s, int t) {
  const int4 g0 = __ldg(reinterpret_cast<const int4*>(gates + s));        // scores ptr, stride, col
  const int4 g1 = __ldg(reinterpret_cast<const int4*>(gates + s) + 1);    // cmp, thr
  const float* sc = reinterpret_cast<const float*>(((unsigned long long)(unsigned)g0.y << 32) | (unsigned)g0.x);
  const float v = __ldg(sc + (size_t)t * g0.z + g0.w);
  const float thr = __int_as_float(g1.y);
  return g1.x == MIX_GATE_GE ? v >= thr : v < thr;
}

// Slot -> app for row t; flags bad slot ids; applies the slot's gate.  `leader` is the one
// thread that may raise status.
__device__ __forceinline__ RowApp lookup(int s, int t, const AppEntry* __restrict__ apps,
                                         const GateEntry* __restrict__ gates, int n_slots,
                                         unsigned* __restrict__ status, bool leader, bool eval_gate = true) {
  RowApp r;
  r.kind = 0;
  r.raw_kind = 0;
  r.C = 0;
  r.gated = false;
  r.chained = false;
  if (s == -1) return r;
  if (s < -1 || s >= n_slots) {
    if (leader) atomicOr(status, MIX_STATUS_BAD_SLOT);
    return r;
  }
  // the whole 48-byte entry in three independent 16-byte loads (one round trip)
  const int4* e = reinterpret_cast<const int4*>(apps + s);
  const int4 q0 = __ldg(e), q1 = __ldg(e + 1), q2 = __ldg(e + 2);
  if (!q0.x) {                                   // valid
    if (leader) atomicOr(status, MIX_STATUS_BAD_SLOT);
    return r;
  }
  r.gated = (q0.y & kKindGated) != 0;
  r.chained = (q0.y & kKindChained) != 0;
  r.raw_kind = q0.y & kKindMask;
  r.C = q0.z;
  if (eval_gate && r.gated && !gate_open(gates, s, t)) return r;  // gate closed: the row passes through
  r.kind = q0.y & kKindMask;
  r.act = q0.w;
  r.alpha = __int_as_float(q1.x);
  r.W = reinterpret_cast<const uint4*>(((unsigned long long)(unsigned)q2.y << 32) | (unsigned)q2.x);
  r.b = reinterpret_cast<const float*>(((unsigned long long)(unsigned)q2.w << 32) | (unsigned)q2.z);
  return r;
}

}  // namespace mix
