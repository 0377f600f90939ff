"""Asynchronous pipeline training of Sec. III-C: the 1F1B order, weight stashing, vertical sync and
weight aggregation, as a plain event walk and a float64 simulation (test infrastructure only;
shares no code with the CUDA library).

What the paper fixes (Sec. III-C, the three-device example in prose; its figure is not available):
  * a stage first forwards as many batches as there are stages from itself to the end, then a
    backward and a forward pass alternate (on stage 0 of three: F0 F1 F2 B0 F3 B1 F4 B2 F5 B3 F6);
  * a batch is backwarded with the weight version it was forwarded with (1_b^0 after 3_f^1);
  * the weight version starts at 0 and every backward pass adds one;
  * stage i holds n - i concurrent versions; they are aggregated at an interval that is a multiple
    of n - i, and the aggregation adds one to the version: after B2 the version is 3, batch 5 is
    forwarded with it, the versions of 3_f^1, 4_f^2, 5_f^3 are aggregated (version 4), B3 gives 5,
    and batch 6 is forwarded with version 5.
Readings where the paper is silent (each a named argument or a line below):
  * "aggregate" is the arithmetic mean of the n - i stashed versions (weights and BN running
    statistics; the momentum buffer of the optimiser is left as it is); it replaces the latest
    weights, and it happens right after the forward pass that follows the (k * (n - i))-th update,
    when the stash holds exactly the n - i versions the example names; the last stage, with a single
    version, has nothing to aggregate;
  * vertical sync: a batch carries the version id it was given on stage 0; a later stage forwards
    it with its own version of that id, or with its latest version if it has not got that far
    (on the last stage of three, batch 1 is forwarded with version 0 although B0 has made version 1);
  * an update is SGD on the stage's latest weights with the gradient taken at the stashed ones;
  * BN running statistics travel with a weight version: a forward pass updates the statistics of
    the copy it runs with, and the update that follows its backward pass keeps them.
"""
import numpy as np

from .model import OracleModel


def stage_order(n_stages, stage, n_batches):
    """[('F' | 'B', batch)] on `stage` (0-indexed) of an n_stages pipeline, 1F1B rule."""
    warm = min(n_stages - stage, n_batches)
    order = [("F", b) for b in range(warm)]
    nf, nb = warm, 0
    while nb < n_batches:
        order.append(("B", nb))
        nb += 1
        if nf < n_batches:
            order.append(("F", nf))
            nf += 1
    return order


def version_trace(n_stages, stage, n_batches, k=1):
    """Walks stage_order with the version counter of Sec. III-C on a stage taken by itself (every
    forward uses the stage's latest version, as on stage 0).  Returns (forward_version[b],
    version after the backward of b, [b: an aggregation follows the forward of b])."""
    c = n_stages - stage
    ver, updates, done_at = 0, 0, 0
    fwd, after_bwd, agg_after = {}, {}, []
    in_flight = []
    for kind, b in stage_order(n_stages, stage, n_batches):
        if kind == "F":
            fwd[b] = ver
            in_flight.append(b)
            if c > 1 and updates > 0 and updates % (k * c) == 0 and updates != done_at and len(in_flight) == c:
                ver += 1
                done_at = updates
                agg_after.append(b)
        else:
            in_flight.remove(b)
            ver += 1
            updates += 1
            after_bwd[b] = ver
    return [fwd[b] for b in range(n_batches)], [after_bwd[b] for b in range(n_batches)], agg_after


class AsyncPipeline:
    """Float64 simulation of the whole pipeline: per stage the latest weights, the versions it has
    had (by id), and one stashed copy per batch in flight."""

    def __init__(self, layers, cfg, params, state, points, k=1):
        self.layers, self.cfg, self.points, self.k = list(layers), dict(cfg), list(points), k
        self.n = len(points) - 1
        self.master = OracleModel(layers, cfg, params, state, storage="none")      # latest weights of every stage
        self.L = self.master.L
        self.ops = [self.master.ops_of(a, b) for a, b in zip(points[:-1], points[1:])]
        self.ver = [0] * self.n
        self.updates = [0] * self.n
        self.agg_done = [0] * self.n
        self.history = [{0: self._take(s)} for s in range(self.n)]               # version id -> (params, running statistics)
        self.stash = [dict() for _ in range(self.n)]                              # batch -> (params, state, version id)
        self.work = {}                                                            # batch -> model holding its activations
        self.stamp = {}                                                           # batch -> version id given on stage 0
        self.losses = {}
        self.log = []

    def _take(self, s, model=None):
        m = model or self.master
        return ([[a.copy() for a in m.p[i]] for i in self.ops[s]], [[a.copy() for a in m.s[i]] for i in self.ops[s]])

    def _put(self, s, model, snap):
        for i, p, st in zip(self.ops[s], snap[0], snap[1]):
            model.p[i] = [a.copy() for a in p]
            model.s[i] = [a.copy() for a in st]

    def forward(self, s, b, x=None, labels=None, act=None):
        if s == 0:
            self.stamp[b] = self.ver[0]
            self.work[b] = OracleModel(self.layers, self.cfg, self.master.p, self.master.s, storage="none")
        want = min(self.stamp[b], self.ver[s])                                   # vertical sync
        vid = max(v for v in self.history[s] if v <= want)
        w = self.work[b]
        self._put(s, w, self.history[s][vid])
        a, e = self.points[s], self.points[s + 1]
        out = w.forward(a, e, x if s == 0 else act, labels if e == self.L else None)
        self.stash[s][b] = (self._take(s, w), vid)                               # weights as used, statistics as updated
        self.log.append(("F", s, b, vid))
        if e == self.L:
            self.losses[b] = w.loss
        c = self.n - s
        if c > 1 and self.updates[s] > 0 and self.updates[s] % (self.k * c) == 0 and self.updates[s] != self.agg_done[s] and len(self.stash[s]) == c:
            self._aggregate(s)
        return out

    def _aggregate(self, s):
        snaps = [v[0] for v in self.stash[s].values()]
        mean_p = [[np.mean([sn[0][i][j] for sn in snaps], axis=0) for j in range(len(snaps[0][0][i]))] for i in range(len(self.ops[s]))]
        mean_s = [[np.mean([sn[1][i][j] for sn in snaps], axis=0) for j in range(len(snaps[0][1][i]))] for i in range(len(self.ops[s]))]
        self._put(s, self.master, (mean_p, mean_s))
        self.ver[s] += 1
        self.agg_done[s] = self.updates[s]
        self.history[s][self.ver[s]] = self._take(s)
        self.log.append(("A", s, sorted(self.stash[s]), self.ver[s]))

    def backward(self, s, b, grad=None, lr=None):
        w = self.work[b]
        a, e = self.points[s], self.points[s + 1]
        snap, vid = self.stash[s].pop(b)
        gin = w.backward(a, e, grad)                                              # gradient at the stashed weights
        for i in self.ops[s]:
            self.master.g[i] = [g.copy() for g in w.g[i]]
        for i, st in zip(self.ops[s], snap[1]):                                   # the statistics of the version just backwarded
            self.master.s[i] = [v.copy() for v in st]
        self.master.sgd(a, e, lr)                                                 # applied to the latest weights
        self.ver[s] += 1
        self.updates[s] += 1
        self.history[s][self.ver[s]] = self._take(s)
        self.log.append(("B", s, b, vid, self.ver[s]))
        if s == 0:
            del self.work[b]
        return gin

    def run(self, batches, lr=None):
        """batches: [(x, labels)].  Executes every stage's 1F1B order as its inputs become available."""
        nb = len(batches)
        orders = [stage_order(self.n, s, nb) for s in range(self.n)]
        pos = [0] * self.n
        acts, grads = {}, {}
        progress = True
        while progress:
            progress = False
            for s in range(self.n):
                while pos[s] < len(orders[s]):
                    kind, b = orders[s][pos[s]]
                    if kind == "F":
                        if s > 0 and (s - 1, b) not in acts:
                            break
                        out = self.forward(s, b, batches[b][0], batches[b][1], acts.pop((s - 1, b), None))
                        if s + 1 < self.n:
                            acts[(s, b)] = out
                    else:
                        if s + 1 < self.n and (s + 1, b) not in grads:
                            break
                        g = self.backward(s, b, grads.pop((s + 1, b), None), lr)
                        if s > 0:
                            grads[(s, b)] = g
                    pos[s] += 1
                    progress = True
        assert all(p == len(o) for p, o in zip(pos, orders)), "the schedule deadlocked"
        return [self.losses[b] for b in range(nb)]
