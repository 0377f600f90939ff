"""Driver of the asynchronous pipeline of Sec. III-C on one GPU: argument marshalling and the order of calls only;
every pass, update, copy and aggregation runs in the library's kernels.

A weight version of a stage is the set of parameter spans of its units inside one model object.  `master` holds
the latest weights of every stage; every batch in flight has a model of its own (its activations live there, and so
do the weights it was forwarded with: the stash).  Per stage a small pool of models keeps the versions the stage has
had, so that a later stage can forward a batch with the version id the batch was given on stage 0 (vertical sync).
The order of passes on a stage comes from ftp_async_stage_order; a stage runs a pass as soon as the neighbouring
stage has delivered its input (an activation forward, a gradient backward).
"""
from . import ftpipe as F


class AsyncPipeline:
    def __init__(self, layers, cfg, points, params, state, k=1, device="cuda:0"):
        self.layers, self.cfg, self.points, self.k = layers, dict(cfg), list(points), k
        self.n = len(points) - 1
        self.device = device
        self.master = F.Model(layers, cfg, device)
        self.master.load_params(params, state)
        self.L = self.master.L
        self.ver = [0] * self.n
        self.updates = [0] * self.n
        self.agg_done = [0] * self.n
        self.free = []                                         # models not in use (activations + one stashed version each)
        self.work = {}                                         # batch -> model holding its activations and stashed weights
        self.stash_ver = [dict() for _ in range(self.n)]       # stage -> batch -> version id it was forwarded with
        self.stamp = {}
        # version history per stage: version id -> model holding that version of the stage's units
        self.history = [dict() for _ in range(self.n)]
        for s in range(self.n):
            self._remember(s)
        self.losses = {}
        self.log = []

    def _model(self):
        return self.free.pop() if self.free else F.Model(self.layers, self.cfg, self.device)

    def _remember(self, s):
        """Keep the stage's latest weights under its current version id."""
        a, b = self.points[s], self.points[s + 1]
        m = self._model()
        F.ftp_sync_units(m, self.master, a, b, F.SYNC_WEIGHTS | F.SYNC_STATE)
        self.history[s][self.ver[s]] = m

    def forward(self, s, b, x=None, labels=None, act=None, loss=None):
        import torch
        a, e = self.points[s], self.points[s + 1]
        if s == 0:
            self.stamp[b] = self.ver[0]
            self.work[b] = self._model()
        w = self.work[b]
        want = min(self.stamp[b], self.ver[s])                 # vertical sync
        vid = max(v for v in self.history[s] if v <= want)
        F.ftp_sync_units(w, self.history[s][vid], a, e, F.SYNC_WEIGHTS | F.SYNC_STATE)
        for old in [v for v in self.history[s] if v < vid]:    # version ids asked for never go down: older ones are done with
            self.free.append(self.history[s].pop(old))
        out = None
        if e == self.L:
            w.ftp_run_stage_forward(a, e, x if s == 0 else act, None, labels, loss)
        else:
            shp, _ = w.ftp_unit_output_shape(e - 1)
            out = torch.empty(shp, dtype=w.act_dtype, device=self.device)
            w.ftp_run_stage_forward(a, e, x if s == 0 else act, out)
        self.stash_ver[s][b] = vid
        self.log.append(("F", s, b, vid))
        c = self.n - s
        if c > 1 and self.updates[s] > 0 and self.updates[s] % (self.k * c) == 0 and self.updates[s] != self.agg_done[s] and len(self.stash_ver[s]) == c:
            srcs = [self.work[q] for q in self.stash_ver[s]]   # the n - i stashed versions, in the order their batches were forwarded
            F.ftp_aggregate_weights(self.master, srcs, a, e)
            self.ver[s] += 1
            self.agg_done[s] = self.updates[s]
            self._remember(s)
            self.log.append(("A", s, sorted(self.stash_ver[s]), self.ver[s]))
        return out

    def backward(self, s, b, grad_out=None, lr=None):
        import torch
        a, e = self.points[s], self.points[s + 1]
        w = self.work[b]
        vid = self.stash_ver[s].pop(b)
        gin = None
        if a > 0:
            shp, _ = w.ftp_unit_output_shape(a - 1)
            gin = torch.empty(shp, dtype=w.act_dtype, device=self.device)
        w.ftp_run_stage_backward(a, e, grad_out, gin)
        F.ftp_sync_units(self.master, w, a, e, F.SYNC_STATE)   # the statistics of the version just backwarded
        F.ftp_sgd_step_from(self.master, w, a, e, self.cfg["lr"] if lr is None else lr)
        self.ver[s] += 1
        self.updates[s] += 1
        self._remember(s)
        self.log.append(("B", s, b, vid, self.ver[s]))
        if s == 0:
            self.free.append(self.work.pop(b))
        return gin

    def run(self, batches, lr=None):
        """batches: [(x, labels)] device tensors.  Returns the loss of every batch (floats)."""
        import torch
        nb = len(batches)
        orders = [F.ftp_async_stage_order(self.n, s, nb) for s in range(self.n)]
        pos = [0] * self.n
        acts, grads, keep_in = {}, {}, {}
        loss_t = {b: torch.zeros(1, device=self.device) for b in range(nb)}
        progress = True
        while progress:
            progress = False
            for s in range(self.n):
                while pos[s] < len(orders[s]):
                    kind, b = orders[s][pos[s]]
                    if kind == "F":
                        if s > 0 and (s - 1, b) not in acts:
                            break
                        inp = acts.pop((s - 1, b), None)
                        keep_in[(s, b)] = inp if s > 0 else batches[b][0]      # a stage's input stays valid until its backward pass
                        out = self.forward(s, b, batches[b][0], batches[b][1], inp, loss_t[b])
                        if s + 1 < self.n:
                            acts[(s, b)] = out
                    else:
                        if s + 1 < self.n and (s + 1, b) not in grads:
                            break
                        g = self.backward(s, b, grads.pop((s + 1, b), None), lr)
                        keep_in.pop((s, b), None)
                        if s > 0:
                            grads[(s, b)] = g
                    pos[s] += 1
                    progress = True
        if not all(p == len(o) for p, o in zip(pos, orders)):
            raise RuntimeError("the schedule deadlocked")
        torch.cuda.synchronize()
        return [float(loss_t[b].item()) for b in range(nb)]

    def close(self):
        for m in [self.master] + self.free + list(self.work.values()) + [m for h in self.history for m in h.values()]:
            m.close()
