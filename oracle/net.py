"""One training step of Algorithm 1 composed from the oracle's layer ops (test infrastructure).

Forward over the layers, integer loss gradient, then the reverse loop: for each layer the
weight gradient and the propagated error are both computed from the layer's incoming error
and its weights *before* the update; the first layer propagates no error.  ReLU and 2x2
max-pool act on the rounded int8 tensors and leave exponents unchanged.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import ref


@dataclass
class OracleNetState:
    weights: list                       # int8 arrays, updated in place of the list entries
    log: list = field(default_factory=list)   # per step: dict of scalars (b values, exponents)


def oracle_train_step(net, x, labels, state: OracleNetState, round_mode=ref.ROUND_PSR,
                      keep_tensors=False, allow_overflow=False):
    """Runs one step; updates ``state.weights``; returns a dict with the scalars of the step
    (and every intermediate tensor when ``keep_tensors``)."""
    acts = []          # input of every layer (post ReLU / pool of the previous one)
    rec = {"b_fwd": [], "s_act": [], "b_e": [], "b_g": []}
    tens = {"act": [], "e": [], "g": []}
    a, s_a = x, net.s_in
    wi = 0
    for L in net.layers:
        acts.append(a)
        if L["op"] == "conv":
            a, s_a, b = ref.conv_fwd(a, s_a, state.weights[wi], L["s_w"], 1, L["relu"], round_mode,
                                     allow_overflow)
            wi += 1
        elif L["op"] == "fc":
            a2 = a.reshape(a.shape[0], -1)
            a, s_a, b = ref.linear_fwd(a2, s_a, state.weights[wi], L["s_w"], L["relu"], round_mode,
                                       allow_overflow)
            wi += 1
        else:
            a = ref.maxpool2_fwd(a)
            b = -1
        rec["b_fwd"].append(b)
        rec["s_act"].append(s_a)
        if keep_tensors:
            tens["act"].append(a)
    e, b_loss, n_correct = ref.int_xent(a, s_a, labels, round_mode)
    rec["b_loss"] = b_loss
    rec["n_correct"] = n_correct
    rec["s_out"] = s_a
    if keep_tensors:
        tens["logits"] = a
        tens["e_loss"] = e
    # reverse loop
    first_weight_layer = next(i for i, L in enumerate(net.layers) if L["op"] != "pool")
    for li in range(len(net.layers) - 1, -1, -1):
        L = net.layers[li]
        a_in = acts[li]
        if L["op"] == "pool":
            # a_in is the ReLU output that was pooled: route to the arg-max, then ReLU mask
            e = ref.maxpool2_bwd(a_in, e.reshape(a_in.shape[0], a_in.shape[1] // 2,
                                                 a_in.shape[2] // 2, a_in.shape[3]))
            if li > 0 and net.layers[li - 1].get("relu"):
                e = ref.relu_bwd(a_in, e)
            continue
        wi -= 1
        w = state.weights[wi]
        need_e = li != first_weight_layer
        # the layer below is ReLU'd iff its output (our input) went through a ReLU and was not
        # pooled in between (pool backward applies the mask itself)
        mask = None
        if need_e and net.layers[li - 1]["op"] != "pool" and net.layers[li - 1].get("relu"):
            mask = a_in
        if L["op"] == "conv":
            g, b_g = ref.conv_wgrad(a_in, e, (3, 3), 1, net.m_u, round_mode, allow_overflow)
            if need_e:
                e_prev, b_e = ref.conv_dgrad(e, w, a_in.shape[1:3], 1, mask, round_mode,
                                             allow_overflow)
            else:
                e_prev, b_e = None, -1
        else:
            a2 = a_in.reshape(a_in.shape[0], -1)
            m2 = None if mask is None else mask.reshape(a2.shape)
            e_prev, g, b_e, b_g = ref.linear_bwd(a2, e.reshape(a2.shape[0], -1), w, need_e, m2,
                                                 net.m_u, round_mode, allow_overflow)
            if e_prev is not None:
                e_prev = e_prev.reshape(a_in.shape)
            else:
                b_e = -1
        rec["b_e"].append(b_e)
        rec["b_g"].append(b_g)
        if keep_tensors:
            tens["g"].append(g)
            tens["e"].append(e_prev)
        state.weights[wi] = ref.sgd_update(w, g)
        e = e_prev
    state.log.append(rec)
    if keep_tensors:
        rec = dict(rec)
        rec["tensors"] = tens
    return rec
