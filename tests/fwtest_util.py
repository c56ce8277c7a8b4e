"""Helpers shared by the GPU parity tests: run the oracle and the CUDA path on
the same seeded inputs and compare, replaying near-tie decisions."""
import copy

import numpy as np

from oracle import fw_oracle as O

TOL_FP32 = 1e-5    # relative Frobenius error bound for the fp32 (FFMA) engine
TOL_TC = 5e-3      # bound for the TF32 / BF16 tensor-core engines
NEAR_TIE = 1e-4    # relative margin below which a discrete decision may legitimately flip (fp32 state)
# With a tensor-core engine the covariance itself differs from the oracle's by up to TOL_TC, and set membership
# is ill-conditioned in it: c_m = <Phi_y e_m, Phi_y e_m'> is compared with c_rel xi_m xi_m', so a relative
# perturbation eps of the columns moves c_m by up to 2 eps / c_rel = 40 eps of its threshold.  The decisions of
# such a layer are therefore checked where they are well defined: on the device's own Phi_y, evaluated by the
# oracle's decision routine in fp64, where only rounding of the fp32 dot products separates the two (margin
# below NEAR_TIE_DEV); the continuous quantities are still compared with the oracle's own state.
NEAR_TIE_DEV = 1e-3
NEAR_TIE_TC = NEAR_TIE_DEV


def rel_fro(a, ref):
    return O.rel_fro(a, ref)


def phiy_error_tc(Py, Lo):
    """Error of a tensor-core layer's Phi_y = T Phi_x T^T, relative to the forward-error scale of the product,
    || |T| |Phi_x| |T|^T ||_F.  A tensor-core Phi_x carries the engine's error (TF32 inputs; fp32 accumulation in
    the tensor core over tens of thousands of rows), and the re-sync multiplies T and Phi_x rounded to TF32: both
    perturb the product by up to tol || |T| |Phi_x| |T|^T ||.  Once the recursion has cut the dominant
    eigenvalues, || Phi_y || is a fraction of that scale (the product cancels), so the same perturbation is a
    larger fraction of || Phi_y ||.  Phi_x, T, Q, Qs and everything downstream stay on the strict relative bound."""
    scale = np.linalg.norm(np.abs(Lo.T) @ np.abs(Lo.Phix) @ np.abs(Lo.T).T)
    return float(np.linalg.norm(Py - Lo.phiy()) / scale)


def t2n(t):
    return t.detach().cpu().numpy().astype(np.float64)


def oracle_hyper(desc):
    return O.Hyper(alpha=desc.alpha, beta=desc.beta, gamma=desc.gamma, delta=desc.delta, eps=desc.eps,
                   c_rel=desc.c_rel, c_abs=desc.c_abs, init=desc.init)


def _check_decisions(Phiy, hp, g_m, g_mask, near_tie, where):
    """The GPU's decisions (g_m, g_mask) against the oracle's decision routine on the matrix Phiy: every
    difference must be a near-tie (relative margin below near_tie)."""
    Phiy = 0.5 * (Phiy + Phiy.T)
    est = O.principal_subspace(Phiy, hp.c_rel, hp.c_abs, hp.init)
    if est["m_prime"] != g_m:
        assert est["margin_argmax"] < near_tie, f"{where}: argmax differs with margin {est['margin_argmax']}"
    if hp.init != O.INIT_MAXCOL:
        est = O.principal_subspace(Phiy, hp.c_rel, hp.c_abs, hp.init, forced=(g_m, None))
        flipped = est["mask"] != g_mask
        worst = float(est["margin_each"][flipped].max()) if flipped.any() else 0.0
        assert worst < near_tie, f"{where}: coherent set differs beyond near-ties (margin {worst})"


def oracle_step_with_replay(ora_layer, g_m, g_mask, P, near_tie, where="", dev_phiy=None):
    """One oracle step that takes its own discrete decisions (m', coherent set)
    unless they differ from the GPU's (g_m, g_mask).  Where they differ, every
    differing decision must be a near-tie (relative margin below near_tie) --
    anything else is a failure -- and the step is re-run with the GPU's
    decisions forced, so the oracle's state stays its own arithmetic.
    The near-tie is judged on the oracle's own Phi_y, or, when dev_phiy (the
    device's Phi_y before the step) is given, on that matrix: the rule for
    tensor-core engines, see NEAR_TIE_DEV.  Returns (trace record, replayed?)."""
    if dev_phiy is not None:
        _check_decisions(dev_phiy, ora_layer.hp, g_m, g_mask, near_tie, where)
    trial = copy.deepcopy(ora_layer)
    rec = O.cond_reduce(trial, 1, P)[0]
    maxcol = ora_layer.hp.init == O.INIT_MAXCOL
    same = rec["m_prime"] == g_m and (maxcol or np.array_equal(rec["mask"], g_mask))
    if same:
        ora_layer.__dict__.update(trial.__dict__)
        return rec, False
    if dev_phiy is None:
        _check_decisions(ora_layer.phiy(), ora_layer.hp, g_m, g_mask, near_tie, where)
    trial2 = copy.deepcopy(ora_layer)
    rec = O.cond_reduce(trial2, 1, P, forced=[(g_m, g_mask)])[0]
    ora_layer.__dict__.update(trial2.__dict__)
    return rec, True


def reduce_with_replay(gpu_layer, ora_layer, K, P, B, torch, near_tie=NEAR_TIE, on_device_state=False):
    """Runs K steps on both sides one step at a time.  After each GPU step its
    discrete decisions (m', coherent set) are read back; the oracle takes its
    own decisions unless they differ from the GPU's on a near-tie, in which case
    the GPU's are replayed (oracle_step_with_replay; on_device_state selects the
    tensor-core rule).  Returns the list of oracle trace records and the number
    of replayed steps."""
    replayed = 0
    records = []
    trace = torch.zeros(4, dtype=torch.float32, device="cuda")
    for k in range(K):
        dev_phiy = t2n(gpu_layer.get(B.FW_F_PHIY)) if on_device_state else None
        gpu_layer.cond_reduce(1, P, trace)
        w = t2n(gpu_layer.get(B.FW_F_ALIGN_W))
        tr = t2n(trace)
        g_m, g_mask = int(round(tr[3])), (w != 0.0)
        rec, rp = oracle_step_with_replay(ora_layer, g_m, g_mask, P, near_tie, f"step {k}", dev_phiy)
        replayed += int(rp)
        rec["gpu_trace"] = tr.copy()
        records.append(rec)
    return records, replayed


def group_reduce_with_replay(gpu_layers, ora_layers, K, P, B, torch, near_tie=NEAR_TIE, on_device_state=False):
    """The grouped form: K grouped calls of one step each over all layers (the
    launch shape of a grouped call: every layer of the group in the same
    launches), each followed by the per-layer decision check and replay of
    reduce_with_replay.  Returns per layer the list of trace records, and the
    total number of replayed steps."""
    hs = [L.handle for L in gpu_layers]
    traces = [torch.zeros(4, dtype=torch.float32, device="cuda") for _ in gpu_layers]
    records = [[] for _ in gpu_layers]
    replayed = 0
    for k in range(K):
        if on_device_state and k == 0:
            B.fw_group_cond_reduce(hs, 0, P)      # the grouped re-sync of Phi_y, as a call with K > 0 starts with
        dev_phiy = [t2n(L.get(B.FW_F_PHIY)) if on_device_state else None for L in gpu_layers]
        B.fw_group_cond_reduce(hs, 1, P, traces)
        for i, (L, Lo) in enumerate(zip(gpu_layers, ora_layers)):
            w = t2n(L.get(B.FW_F_ALIGN_W))
            tr = t2n(traces[i])
            g_m, g_mask = int(round(tr[3])), (w != 0.0)
            rec, rp = oracle_step_with_replay(Lo, g_m, g_mask, P, near_tie, f"layer {i} step {k}", dev_phiy[i])
            replayed += int(rp)
            rec["gpu_trace"] = tr.copy()
            records[i].append(rec)
    return records, replayed
