"""The paper's rollout stage-time model (Appendix A.1, "Rollout Model") as a CPU utility, with its
decode-history coefficient tied to libpdattn's measured bandwidth.

The model predicts the time one rollout replica needs for a set of requests with prompt lengths p_i
and response lengths r_i, and M_r(n, d) = max over replicas (the replica-max rule).  Its decode part is

    P_dec = tau_dec * W_dec + beta_tok * N_tok + beta_hist * H_dec,

where H_dec = sum_i (r_i p_i + r_i (r_i - 1) / 2) counts the history tokens attention reads.  Decode
attention is bandwidth bound, so beta_hist is what this library measures: reading one history token
costs b_kv bytes (all layers), hence beta_hist = b_kv / (achieved KV bytes per second).

Vectorised with numpy (decode steps are handled through sorted response lengths, not a loop over
requests); the plain-loop statement of the same formulas lives with the tests.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Sequence

import numpy as np


@dataclasses.dataclass
class RolloutModel:
    """Constants of the rollout model, in the paper's notation."""
    L: int                  # layers
    H_kv: int               # KV heads
    d_head: int
    H: int                  # hidden size
    V: int                  # vocabulary size
    N_nonemb: float         # non-embedding parameters
    B_kv: float             # KV-cache budget of a replica, bytes
    b_dtype: int = 2
    tp: int = 1
    tau_pre: float = 0.0    # per prefill wave
    alpha_pre: float = 0.0  # per prefill FLOP
    tau_dec: float = 0.0    # per decode wave
    beta_tok: float = 0.0   # per generated token
    beta_hist: float = 0.0  # per history token read
    C_pre: float = 0.0      # communication terms of the two phases
    C_dec: float = 0.0
    r: float = 1.0          # overlap exponent

    @property
    def b_kv(self) -> float:
        """per-token KV-cache footprint 2 L H_kv d_head b_dtype / tp"""
        return 2.0 * self.L * self.H_kv * self.d_head * self.b_dtype / self.tp

    def N_max(self, ell: float) -> int:
        """KV-limited concurrency at average live length ell"""
        return max(1, int(math.floor(self.B_kv / (self.b_kv * ell))))

    def with_measured_bandwidth(self, kv_bytes_per_second: float) -> "RolloutModel":
        """beta_hist from a measured decode-attention bandwidth (bytes of KV read per second)."""
        return dataclasses.replace(self, beta_hist=self.b_kv / kv_bytes_per_second)

    # ---- features -------------------------------------------------------------------------------
    def prefill_features(self, p: Sequence[int]):
        p = np.asarray(p, dtype=np.float64)
        B_j = p.size
        N_pre = min(B_j, self.N_max(float(p.mean())))
        W_pre = -(-B_j // N_pre)
        F_pre = 2.0 * self.N_nonemb * p.sum() + 4.0 * self.L * self.H * np.square(p).sum() + 2.0 * self.H * self.V * B_j
        return N_pre, W_pre, float(F_pre)

    def decode_features(self, p: Sequence[int], r: Sequence[int]):
        p = np.asarray(p, dtype=np.int64)
        r = np.asarray(r, dtype=np.int64)
        N_tok = int(r.sum())
        H_dec = int((r * p + r * (r - 1) // 2).sum())
        if r.size == 0 or r.max() <= 0:
            return 0, N_tok, H_dec
        # live set of step t = requests with r_i >= t: a suffix of the requests sorted by r
        order = np.argsort(r, kind="stable")
        rs, ps = r[order], p[order]
        suffix_p = np.concatenate([np.cumsum(ps[::-1])[::-1], [0]])
        t = np.arange(1, int(rs[-1]) + 1)
        first = np.searchsorted(rs, t, side="left")              # first sorted index with r >= t
        n_live = r.size - first
        ell = suffix_p[first] / n_live + (t - 1)
        n_max = np.maximum(1, np.floor(self.B_kv / (self.b_kv * ell))).astype(np.int64)
        w = -(-n_live // np.minimum(n_live, n_max))
        return int(w.sum()), N_tok, H_dec

    # ---- times ------------------------------------------------------------------------------------
    @staticmethod
    def overlap(x: float, c: float, r: float) -> float:
        return (x ** r + c ** r) ** (1.0 / r)

    def T_r_rep(self, p: Sequence[int], r: Sequence[int]) -> float:
        """time of one replica for its requests"""
        if len(p) == 0:
            return 0.0
        _, W_pre, F_pre = self.prefill_features(p)
        W_dec, N_tok, H_dec = self.decode_features(p, r)
        P_pre = self.tau_pre * W_pre + self.alpha_pre * F_pre
        P_dec = self.tau_dec * W_dec + self.beta_tok * N_tok + self.beta_hist * H_dec
        return self.overlap(P_pre, self.C_pre, self.r) + self.overlap(P_dec, self.C_dec, self.r)

    def M_r(self, prompts: Sequence[int], responses: Sequence[Sequence[int]], d: int) -> float:
        """stage time of d replicas for n prompt-level groups (prompt k with its sampled response
        lengths responses[k]); group k goes to replica k mod d; the slowest replica decides."""
        worst = 0.0
        for j in range(d):
            p, r = [], []
            for k in range(j, len(prompts), d):
                p.extend([prompts[k]] * len(responses[k]))
                r.extend(responses[k])
            worst = max(worst, self.T_r_rep(p, r))
        return worst
