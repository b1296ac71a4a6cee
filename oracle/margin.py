"""Input repair for bit-exact index sets (TEST INFRASTRUCTURE; calls the oracle).

The retention rule s_t >= tau (Sec. 3.2) turns a float into a decision.  So that the CUDA path and
the oracle take the same decision for every chunk, the seeded inputs are adjusted until no score
lies within `margin` of tau: the oracle's gate is run chunk by chunk in temporal order; a chunk of
a sequence whose score falls inside the band is redrawn from a sub-seed (workload seed, layer,
sequence, chunk, attempt) and its step recomputed.  Because the LSTM is causal (Eq. 3), earlier
scores are not touched by a redraw.
"""
import numpy as np

from paper_2509_21354_b200 import workloads as wlm

from . import kvo

AGG_CODE = {"mean": kvo.AGG_MEAN, "mlp": kvo.AGG_MLP, "identity": kvo.AGG_IDENTITY, "max": kvo.AGG_MAX,
            "token_mlp": kvo.AGG_TOKEN_MLP}


def centred_b_s(o: kvo.Oracle, wl: wlm.Workload, K, V, mlp, lstm, keep=0.5, n_chunks=None):
    """Head bias that puts the (1 - keep) quantile of the score logits at tau: with it about `keep`
    of the chunks are retained.  Deterministic given the seeded inputs."""
    S, n, d = K.shape
    Nc = wl.n_stale_chunks(n) if n_chunks is None else n_chunks
    if Nc == 0:
        return 0.0
    sm = o.summarize(K, V, wl.C, 0, Nc, AGG_CODE[wl.agg], mlp, stride=Nc)
    z = dict(lstm)
    z["b_s"] = 0.0
    sc, _, _ = o.gate(sm["ksum_b16"], sm["vsum_b16"], 0, Nc, z)
    sc = np.clip(sc[:, :Nc].astype(np.float64), 1e-12, 1 - 1e-12)
    logit = np.log(sc / (1 - sc))
    t = np.log(wl.tau / (1 - wl.tau))
    return float(t - np.quantile(logit, 1.0 - keep))


def repair_margin(o: kvo.Oracle, wl: wlm.Workload, layer, K, V, mlp, lstm, tau=None, margin=1e-3,
                  n_chunks=None, max_attempts=50, seq_ids=None):
    """Adjusts K, V in place.  Returns (summaries dict, scores [S, stride], h, c, redraws) as the
    oracle `o` computes them on the repaired inputs; redraws = [(s, t, attempt), ...].
    K, V may hold a subset of the workload's sequences: seq_ids[i] is the sequence id of row i."""
    tau = wl.tau if tau is None else tau
    S, n, d = K.shape
    seq_ids = list(range(S)) if seq_ids is None else [int(x) for x in seq_ids]
    Nc = wl.n_stale_chunks(n) if n_chunks is None else n_chunks
    stride = max(wl.max_chunks, 1)
    agg = AGG_CODE[wl.agg]
    sm = dict(ksum=np.zeros((S, stride, d), o.real), vsum=np.zeros((S, stride, d), o.real),
              ksum_b16=np.zeros((S, stride, d), np.uint16), vsum_b16=np.zeros((S, stride, d), np.uint16))
    if Nc > 0:
        o.summarize(K, V, wl.C, 0, Nc, agg, mlp, stride=stride, out=sm)
    h = np.zeros((S, wl.d_g), o.real)
    c = np.zeros((S, wl.d_g), o.real)
    scores = np.zeros((S, stride), o.real)
    redraws = []
    for t in range(Nc):
        h0, c0 = h.copy(), c.copy()
        o.gate(sm["ksum_b16"], sm["vsum_b16"], t, t + 1, lstm, h, c, scores)
        bad = np.nonzero(np.abs(scores[:, t].astype(np.float64) - tau) < margin)[0]
        attempt = {int(s): 0 for s in bad}
        while len(bad):
            for s in bad:
                s = int(s)
                attempt[s] += 1
                if attempt[s] > max_attempts:
                    raise RuntimeError("margin repair did not converge")
                k, v = wlm.gen_chunk(wl, layer, seq_ids[s], t, attempt[s])
                K[s, t * wl.C:(t + 1) * wl.C] = k
                V[s, t * wl.C:(t + 1) * wl.C] = v
            # re-summarise and re-gate just the redrawn (sequence, chunk) pairs from the saved state
            Kb = np.ascontiguousarray(K[bad, t * wl.C:(t + 1) * wl.C])
            Vb = np.ascontiguousarray(V[bad, t * wl.C:(t + 1) * wl.C])
            one = o.summarize(Kb, Vb, wl.C, 0, 1, agg, mlp, stride=1)
            hb, cb = np.ascontiguousarray(h0[bad]), np.ascontiguousarray(c0[bad])
            sb, hb, cb = o.gate(one["ksum_b16"], one["vsum_b16"], 0, 1, lstm, hb, cb)
            for key in sm:
                sm[key][bad, t] = one[key][:, 0]
            h[bad], c[bad], scores[bad, t] = hb, cb, sb[:, 0]
            still = np.abs(sb[:, 0].astype(np.float64) - tau) < margin
            bad = bad[still]
        redraws.extend((seq_ids[s], t, a) for s, a in attempt.items())
    return sm, scores, h, c, redraws
