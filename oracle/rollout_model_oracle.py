"""TEST INFRASTRUCTURE: the paper's rollout stage-time model (Appendix A.1, "Rollout Model" and the
replica-max rule) written out with plain Python loops, one function per printed formula, in the paper's
notation.  It checks paper_2607_09207_b200/rollout_model.py and shares no code with it.

Pins (tests/test_rollout_model.py): hand-evaluated cases in tests/golden/rollout_model.txt, closed forms
(H_dec of equal requests, W_dec when the cache never limits concurrency, overlap limits r = 1 and r -> inf).
"""
import math


def b_kv(L, H_kv, d_head, b_dtype, tp):
    """per-token KV-cache footprint: 2 L H_kv d_head b_dtype / tp"""
    return 2.0 * L * H_kv * d_head * b_dtype / tp


def N_max(B_kv, bkv, ell):
    """KV-limited concurrency at average live length ell: max(1, floor(B_kv / (b_kv ell)))"""
    return max(1, int(math.floor(B_kv / (bkv * ell))))


def overlap(x, c, r):
    """p-norm overlap of compute x and communication c: (x^r + c^r)^(1/r)"""
    return (x ** r + c ** r) ** (1.0 / r)


def prefill_features(p, B_kv, bkv, N_nonemb, L, H, V):
    """(N_pre, W_pre, F_pre) for the requests with prompt lengths p"""
    B_j = len(p)
    mean_p = sum(p) / B_j
    N_pre = min(B_j, N_max(B_kv, bkv, mean_p))
    W_pre = int(math.ceil(B_j / N_pre))
    F_pre = 2.0 * N_nonemb * sum(p) + 4.0 * L * H * sum(x * x for x in p) + 2.0 * H * V * B_j
    return N_pre, W_pre, F_pre


def decode_features(p, r, B_kv, bkv):
    """(W_dec, N_tok, H_dec): decode step t has live set A_t = {i : r_i >= t}, mean live length
    ell_t = mean_{A_t}(p_i + t - 1) and w_t = ceil(|A_t| / min(|A_t|, N_max(ell_t))) waves."""
    W_dec = 0
    t = 1
    while True:
        A_t = [i for i in range(len(r)) if r[i] >= t]
        if not A_t:
            break
        ell_t = sum(p[i] + t - 1 for i in A_t) / len(A_t)
        w_t = int(math.ceil(len(A_t) / min(len(A_t), N_max(B_kv, bkv, ell_t))))
        W_dec += w_t
        t += 1
    N_tok = sum(r)
    H_dec = sum(r[i] * p[i] + r[i] * (r[i] - 1) // 2 for i in range(len(r)))
    return W_dec, N_tok, H_dec


def T_r_rep(p, r, c):
    """rollout replica time: overlap(P_pre, C_pre, r) + overlap(P_dec, C_dec, r) with
    P_pre = tau_pre W_pre + alpha_pre F_pre and P_dec = tau_dec W_dec + beta_tok N_tok + beta_hist H_dec.
    c: dict of the model's constants."""
    if not p:
        return 0.0
    bkv = b_kv(c["L"], c["H_kv"], c["d_head"], c["b_dtype"], c["tp"])
    _, W_pre, F_pre = prefill_features(p, c["B_kv"], bkv, c["N_nonemb"], c["L"], c["H"], c["V"])
    P_pre = c["tau_pre"] * W_pre + c["alpha_pre"] * F_pre
    W_dec, N_tok, H_dec = decode_features(p, r, c["B_kv"], bkv)
    P_dec = c["tau_dec"] * W_dec + c["beta_tok"] * N_tok + c["beta_hist"] * H_dec
    return overlap(P_pre, c["C_pre"], c["r"]) + overlap(P_dec, c["C_dec"], c["r"])


def M_r(groups, d, c):
    """replica-max rule: prompt-level groups are dealt to the d replicas in turn (group k to replica
    k mod d); the stage time is the slowest replica.  groups: list of (p, [r_1..r_m]) per prompt."""
    worst = 0.0
    for j in range(d):
        p, r = [], []
        for k in range(j, len(groups), d):
            for ri in groups[k][1]:
                p.append(groups[k][0])
                r.append(ri)
        worst = max(worst, T_r_rep(p, r, c))
    return worst
