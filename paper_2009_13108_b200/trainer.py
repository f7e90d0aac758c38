"""One integer training step (Algorithm 1 of the paper) as a fixed sequence of library calls.

All tensors are allocated once; a step enqueues kernels on the current stream and never
synchronises with the host, so it can be captured in a CUDA graph.  ReLU is fused into the
forward epilogue, the ReLU mask into the dgrad epilogue, and the ReLU mask of a pooled layer
into the max-pool backward."""
from __future__ import annotations

import torch

from .api import Niti, ROUND_PSR


class NitiTrainer:
    def __init__(self, niti: Niti, net, weights, round_mode: int = ROUND_PSR, fused_update: bool = True,
                 pool_codes: bool = False, dist_group=None, data_parallel: bool = False, pool_fused: bool = True):
        """``net``: an object with ``batch``, ``in_shape``, ``s_in``, ``m_u`` and ``layers`` (dicts
        with op in {"conv", "pool", "fc"}); ``weights``: int8 host arrays / tensors per weight
        layer ([Cout,3,3,Cin] or [N,K]).  ``fused_update``: weight gradient and weight update in one
        library call (Section 3.3), else ``*_wgrad`` / ``linear_bwd`` followed by ``int_sgd_update``;
        the weights after a step are the same either way.  The fused calls compute the error of the
        layer below first (it needs the old weights) and never store the int8 gradient where the
        rounding pass can subtract from the weights directly; measured 0.5 % faster on VGG-16.
        ``pool_codes``: the max-pool forward records
        its routing (half a byte per output element) and the backward pass reads that instead of the
        pooled tensor; in isolation the backward kernels get 30 % faster and the forward ones 15-40 %
        slower, over the VGG-16 step it measured 0.5 % slower, so it is off by default."""
        self.n = niti
        self.net = net
        self.round_mode = round_mode
        self.fused_update = fused_update
        # ``pool_fused``: a convolution that is followed by a max-pool writes the pooled tensor from its own
        # epilogue (niti_conv_fwd_pool) and the separate pooling pass of the forward step is dropped
        self.pool_fused = pool_fused and not pool_codes
        # exact data parallelism: ``net.batch`` is this rank's share of the batch; bit-widths and
        # weight-gradient sums are combined over the ranks of ``dist_group`` (None = the default group),
        # so every rank holds the weights one process with the whole batch would have
        self.data_parallel = data_parallel
        if data_parallel:
            import torch.distributed as dist
            from .api import dist_reducer
            niti.set_reduce_hook(dist_reducer(dist_group))
            # weight gradients: reduce-scatter of the int32 sums, per-shard rounding, all-gather of int8
            niti.set_dp_shard(dist.get_rank(dist_group), dist.get_world_size(dist_group))
            self._dist_group = dist_group
        dev = niti.device
        i8 = dict(dtype=torch.int8, device=dev)
        self.weights = [torch.as_tensor(w).to(dev).contiguous() for w in weights]
        self._initial = None
        self.s_in = niti.scalar(net.s_in)
        self.x = torch.empty((net.batch,) + tuple(net.in_shape), **i8)
        self.labels = torch.empty((net.batch,), dtype=torch.int32, device=dev)
        # forward buffers
        self.acts, self.s_act, self.b_fwd, self.s_w, self.pool_idx = [], [], [], [], []
        shape = self.x.shape
        wi = 0
        max_act, max_w = 0, 0
        for L in net.layers:
            if L["op"] == "conv":
                shape = (shape[0], shape[1], shape[2], L["cout"])
            elif L["op"] == "pool":
                shape = (shape[0], shape[1] // 2, shape[2] // 2, shape[3])
            else:
                shape = (shape[0], L["n"])
            self.acts.append(torch.empty(shape, **i8))
            # routing codes of a max-pool (half a byte per output element): its backward pass then
            # reads them instead of the pooled tensor
            self.pool_idx.append(torch.empty(shape[:3] + (shape[3] // 2,), dtype=torch.uint8, device=dev)
                                 if L["op"] == "pool" and shape[3] % 16 == 0 and pool_codes else None)
            self.s_act.append(niti.scalar())
            self.b_fwd.append(niti.scalar(-1))
            if L["op"] != "pool":
                self.s_w.append(niti.scalar(L["s_w"]))
                max_w = max(max_w, self.weights[wi].numel())
                wi += 1
            else:
                self.s_w.append(None)
            max_act = max(max_act, self.acts[-1].numel())
        max_act = max(max_act, self.x.numel())
        # backward buffers: two ping-pong error buffers and one gradient buffer
        self.e_buf = [torch.empty(max_act, **i8), torch.empty(max_act, **i8)]
        self.g_buf = torch.empty(max_w, **i8)
        self.b_e = [niti.scalar(-1) for _ in net.layers]
        self.b_g = [niti.scalar(-1) for _ in net.layers]
        self.b_loss = niti.scalar()
        self.n_correct = niti.scalar()
        self.first_weight_layer = next(i for i, L in enumerate(net.layers) if L["op"] != "pool")
        # an image network's first convolution (1 or 3 input channels) gathers its taps once per step: the
        # weight gradient at the end of the step reads the rows the forward pass gathered
        L0 = net.layers[self.first_weight_layer]
        if L0["op"] == "conv" and 9 * L0["cin"] <= 32 and L0["cin"] % 16 != 0:
            niti.set_tap_cache(32 * self.acts[self.first_weight_layer].numel() // L0["cout"])

    def global_hits(self):
        """Hit count of the last step over all ranks (data parallel), as a device tensor."""
        hits = self.n_correct.clone()
        if self.data_parallel:
            import torch.distributed as dist
            dist.all_reduce(hits, op=dist.ReduceOp.SUM, group=self._dist_group)
        return hits

    def snapshot_weights(self):
        """Keeps a device copy of the current weights for reset_weights()."""
        self._initial = [w.clone() for w in self.weights]

    def reset_weights(self):
        """Restores the snapshot (device-to-device copies on the current stream)."""
        for w, w0 in zip(self.weights, self._initial):
            w.copy_(w0, non_blocking=True)

    def capture(self, with_reset: bool = False):
        """Captures one step (optionally preceded by reset_weights) into a CUDA graph; returns a
        callable that replays it on the current stream.  Run at least one eager step first: the
        library sizes its kernel attributes on first use, which must happen outside a capture."""
        stream = torch.cuda.Stream(device=self.n.device)
        stream.wait_stream(torch.cuda.current_stream(self.n.device))
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(graph, stream=stream):
                if with_reset:
                    self.reset_weights()
                self.step()
        torch.cuda.current_stream(self.n.device).wait_stream(stream)
        self._graph = graph
        return graph.replay

    def load_batch(self, x, labels):
        """Copies one batch (host or device tensors) into the resident input buffers."""
        self.x.copy_(torch.as_tensor(x).reshape(self.x.shape), non_blocking=True)
        self.labels.copy_(torch.as_tensor(labels), non_blocking=True)

    def prefetch_batch(self, x, labels):
        """Starts the host-to-device copy of the NEXT batch (pinned host tensors) on a copy stream
        into staging buffers, so that it overlaps the step running on the current stream;
        ``commit_batch`` makes it the current batch."""
        dev = self.n.device
        if not hasattr(self, "_copy_stream"):
            self._copy_stream = torch.cuda.Stream(device=dev)
            self._x_stage = torch.empty_like(self.x)
            self._labels_stage = torch.empty_like(self.labels)
            self._staged = torch.cuda.Event()
            self._stage_free = torch.cuda.Event()
            self._stage_free.record(torch.cuda.current_stream(dev))
        self._copy_stream.wait_event(self._stage_free)       # the previous commit has read the staging buffers
        with torch.cuda.stream(self._copy_stream):
            self._x_stage.copy_(torch.as_tensor(x).reshape(self.x.shape), non_blocking=True)
            self._labels_stage.copy_(torch.as_tensor(labels), non_blocking=True)
            self._staged.record(self._copy_stream)

    def commit_batch(self):
        """Makes the prefetched batch the resident one (device-to-device, on the current stream)."""
        cur = torch.cuda.current_stream(self.n.device)
        cur.wait_event(self._staged)
        self.x.copy_(self._x_stage, non_blocking=True)
        self.labels.copy_(self._labels_stage, non_blocking=True)
        self._stage_free.record(cur)

    def _view(self, buf, shape):
        n = 1
        for d in shape:
            n *= d
        return buf[:n].view(shape)

    def forward(self):
        n, net = self.n, self.net
        a, s = self.x, self.s_in
        wi = 0
        pooled_by_conv = -1
        for li, L in enumerate(net.layers):
            out = self.acts[li]
            if L["op"] == "conv":
                nxt_is_pool = li + 1 < len(net.layers) and net.layers[li + 1]["op"] == "pool"
                if self.pool_fused and nxt_is_pool and L["relu"] and a.shape[1] % 2 == 0 and a.shape[2] % 2 == 0:
                    n.conv_fwd_pool(a, s, self.weights[wi], self.s_w[li], y=out, y_pool=self.acts[li + 1],
                                    s_y=self.s_act[li], b_y=self.b_fwd[li], pad=1, relu=True,
                                    round_mode=self.round_mode)
                    pooled_by_conv = li + 1
                else:
                    n.conv_fwd(a, s, self.weights[wi], self.s_w[li], y=out, s_y=self.s_act[li],
                               b_y=self.b_fwd[li], pad=1, relu=L["relu"], round_mode=self.round_mode)
                s = self.s_act[li]
                wi += 1
            elif L["op"] == "fc":
                n.linear_fwd(a.reshape(a.shape[0], -1), s, self.weights[wi], self.s_w[li], out=out,
                             s_out=self.s_act[li], b_out=self.b_fwd[li], relu=L["relu"],
                             round_mode=self.round_mode)
                s = self.s_act[li]
                wi += 1
            elif pooled_by_conv == li:
                pass                                  # written by the convolution before it
            else:
                if self.pool_idx[li] is not None:
                    n.maxpool2_fwd_idx(a, y=out, idx=self.pool_idx[li])
                else:
                    n.maxpool2_fwd(a, y=out)
            a = out
        return a, s

    def step(self):
        """Forward, integer loss gradient, backward with in-place weight update."""
        n, net = self.n, self.net
        n.begin_step()                     # one memset instead of one per multiply (the workspace is sized by then)
        logits, s_out = self.forward()
        cur = 0
        e = self._view(self.e_buf[cur], logits.shape)
        n.int_xent(logits, s_out, self.labels, e=e, b_e=self.b_loss, n_correct=self.n_correct,
                   round_mode=self.round_mode)
        wi = len(self.weights)
        for li in range(len(net.layers) - 1, -1, -1):
            L = net.layers[li]
            a_in = self.x if li == 0 else self.acts[li - 1]
            if L["op"] == "pool":
                nxt = self._view(self.e_buf[cur ^ 1], a_in.shape)
                relu = bool(li > 0 and net.layers[li - 1].get("relu"))
                if self.pool_idx[li] is not None:
                    n.maxpool2_bwd_idx(e.view(self.acts[li].shape), self.pool_idx[li], a_in.shape, e_in=nxt,
                                       relu=relu)
                else:
                    n.maxpool2_bwd(a_in, e.view(self.acts[li].shape), e_in=nxt, relu=relu)
                e, cur = nxt, cur ^ 1
                continue
            wi -= 1
            w = self.weights[wi]
            need_e = li != self.first_weight_layer
            mask = None
            if need_e and net.layers[li - 1]["op"] != "pool" and net.layers[li - 1].get("relu"):
                mask = a_in
            g = self._view(self.g_buf, w.shape)
            nxt = self._view(self.e_buf[cur ^ 1], a_in.shape) if need_e else None
            if L["op"] == "conv":
                ev = e.view(self.acts[li].shape)
                if self.fused_update:
                    if need_e:                     # from the weights as they are before the update
                        n.conv_dgrad(ev, w, a_in.shape[1:3], e_prev=nxt, relu_mask_src=mask,
                                     b_e=self.b_e[li], pad=1, round_mode=self.round_mode)
                    n.conv_wgrad_update(a_in, ev, w, b_g=self.b_g[li], pad=1, m_u=net.m_u,
                                        round_mode=self.round_mode)
                else:
                    n.conv_wgrad(a_in, ev, (3, 3), g=g, b_g=self.b_g[li], pad=1, m_u=net.m_u,
                                 round_mode=self.round_mode)
                    if need_e:
                        n.conv_dgrad(ev, w, a_in.shape[1:3], e_prev=nxt, relu_mask_src=mask,
                                     b_e=self.b_e[li], pad=1, round_mode=self.round_mode)
                    n.int_sgd_update(w, g)
            else:
                a2 = a_in.reshape(a_in.shape[0], -1)
                kw = dict(need_e_prev=need_e,
                          relu_mask_src=None if mask is None else mask.reshape(a2.shape),
                          e_prev=None if nxt is None else nxt.view(a2.shape),
                          b_e=self.b_e[li], b_g=self.b_g[li], m_u=net.m_u, round_mode=self.round_mode)
                if self.fused_update:
                    n.linear_bwd_update(a2, e.view(a2.shape[0], -1), w, **kw)
                else:
                    n.linear_bwd(a2, e.view(a2.shape[0], -1), w, g=g, **kw)
                    n.int_sgd_update(w, g)
            if need_e:
                e, cur = nxt, cur ^ 1
        return self.n_correct
