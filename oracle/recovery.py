"""Training state of a node and the central node's fault handler, as plain data and functions
(test infrastructure only; shares no code with the CUDA library).

Follows Sec. III-B, Table I (the state variables every node holds and their initial values) and
Sec. III-F (the timer on the central node, `status`, the three outcomes of the probe, the reset
of the committed ids that lets training resume).
"""

NORMAL, RESTARTED, SILENT = 0, 1, 2                 # how a worker answers the handler's probe
RESTART_BATCH, RESEND_STATE, REDISTRIBUTE = 0, 1, 2 # what the handler does next


class TrainState:
    """Table I: committed forward / backward id start at -1, status at 0 (normal; 1 = fault recovery)."""

    def __init__(self, learning_rate, epoch_number, batch_number):
        self.committed_forward_id = -1
        self.committed_backward_id = -1
        self.status = 0
        self.learning_rate = learning_rate
        self.epoch_number = epoch_number
        self.batch_number = batch_number

    def forward_done(self, batch_id):
        """The latest id of the batch that has completed forwarding."""
        self.committed_forward_id = batch_id

    def backward_done(self, batch_id):
        self.committed_backward_id = batch_id

    def timer_expired(self, batch_id):
        """Sec. III-F: the gradients of `batch_id` did not come back in time.  The handler runs once:
        status goes to 1 and later timers find it set.  Returns True when this call triggers it."""
        if self.status == 1:
            return False
        self.status = 1
        return True

    def may_forward(self, batch_id):
        """While recovering, a node stops forwarding batches beyond its committed forward id
        (they were sent before the sub-models were rebuilt and are discarded)."""
        return self.status == 0 or batch_id <= self.committed_forward_id

    def reset(self, batch_id):
        """Last phase of the handler: both committed ids become the id of the batch whose gradients
        were not received, status returns to 0, and training resumes by forwarding that batch."""
        self.committed_forward_id = batch_id
        self.committed_backward_id = batch_id
        self.status = 0
        return batch_id


def classify_probe(responses):
    """Sec. III-F, the three cases of the probe.  responses[i] in {NORMAL, RESTARTED, SILENT} for
    worker i of the worker list (worker 0 is the central node itself and is NORMAL).
      all normal                          -> (RESTART_BATCH, [], None): restart from the lost batch;
      all answer, exactly one restarted   -> (RESEND_STATE, [], w): send worker w the state variables; it
                                             reloads its weights from the replica its neighbour keeps;
      otherwise                           -> (REDISTRIBUTE, failed, None): the silent workers are dropped
                                             from the list (one: Algorithm 1 with its index; several: chain
                                             plus global replicas).  A worker that restarted beside other
                                             faults has lost its weights like a silent one and is counted
                                             as failed (the paper names no separate case for it)."""
    assert responses and responses[0] == NORMAL, "worker 0 is the central node"
    silent = [i for i, r in enumerate(responses) if r == SILENT]
    restarted = [i for i, r in enumerate(responses) if r == RESTARTED]
    if not silent and not restarted:
        return RESTART_BATCH, [], None
    if not silent and len(restarted) == 1:
        return RESEND_STATE, [], restarted[0]
    return REDISTRIBUTE, sorted(silent + restarted), None
