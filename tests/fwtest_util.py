"""Helpers shared by the GPU parity tests: run the oracle and the CUDA path on
the same seeded inputs and compare, replaying near-tie decisions."""
import numpy as np

from oracle import fw_oracle as O

TOL_FP32 = 1e-5    # relative Frobenius error bound for the fp32 (FFMA) engine
TOL_TC = 5e-3      # bound for the TF32 / BF16 tensor-core engines
NEAR_TIE = 1e-4    # relative margin below which a discrete decision may legitimately flip


def rel_fro(a, ref):
    return O.rel_fro(a, ref)


def t2n(t):
    return t.detach().cpu().numpy().astype(np.float64)


def oracle_hyper(desc):
    return O.Hyper(alpha=desc.alpha, beta=desc.beta, gamma=desc.gamma, delta=desc.delta, eps=desc.eps,
                   c_rel=desc.c_rel, c_abs=desc.c_abs, init=desc.init)


def reduce_with_replay(gpu_layer, ora_layer, K, P, B, torch):
    """Runs K steps on both sides one step at a time.  After each GPU step its
    discrete decisions (m', coherent set) are read back; the oracle takes its
    own decisions unless they differ from the GPU's on a near-tie (relative
    margin < NEAR_TIE), in which case the GPU's are replayed.  A difference with
    a larger margin is a failure.  Returns the list of oracle trace records and
    the number of replayed steps."""
    import copy
    replayed = 0
    records = []
    trace = torch.zeros(4, dtype=torch.float32, device="cuda")
    for k in range(K):
        gpu_layer.cond_reduce(1, P, trace)
        w = t2n(gpu_layer.get(B.FW_F_ALIGN_W))
        tr = t2n(trace)
        g_m, g_mask = int(round(tr[3])), (w != 0.0)
        trial = copy.deepcopy(ora_layer)
        rec = O.cond_reduce(trial, 1, P)[0]
        same = rec["m_prime"] == g_m and (ora_layer.hp.init == O.INIT_MAXCOL or np.array_equal(rec["mask"], g_mask))
        if same:
            ora_layer.__dict__.update(trial.__dict__)
        else:
            if rec["m_prime"] != g_m:
                assert rec["margin_argmax"] < NEAR_TIE, f"step {k}: argmax differs with margin {rec['margin_argmax']}"
            trial2 = copy.deepcopy(ora_layer)
            rec = O.cond_reduce(trial2, 1, P, forced=[(g_m, g_mask)])[0]
            if rec["m_prime"] == g_m:
                # set difference: every flipped member must be a near-tie in the oracle
                est = O.principal_subspace(0.5 * (ora_layer.phiy() + ora_layer.phiy().T), ora_layer.hp.c_rel,
                                           ora_layer.hp.c_abs, ora_layer.hp.init, forced=(g_m, None))
                flipped = est["mask"] != g_mask
                assert np.all(est["margin_each"][flipped] < NEAR_TIE), \
                    f"step {k}: coherent set differs beyond near-ties"
            ora_layer.__dict__.update(trial2.__dict__)
            replayed += 1
        rec["gpu_trace"] = tr.copy()
        records.append(rec)
    return records, replayed
