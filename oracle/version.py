"""Model of a rollout worker's policy-version state (oracle side).

Section 4.2 ("Policy publication", "Rollout generation") and Section 4.3: the
learner publishes immutable, versioned snapshots; a worker keeps generating
under its installed snapshot while a newer one arrives, switches its local
version only once the new snapshot is completely installed, and tags each
trajectory with the single version it was generated under (Algorithm 1, rollout
plane: update local version if a newer snapshot is fully installed; then
sample; then push (x, y, r, v)).

With two weight buffers the worker holds at most two versions: the one it
serves and one being installed.  A third offer while an install is pending is
refused ("busy"); versions must strictly increase.

Pins: the state-machine tests replay the sequences of events spelled out above
(overlapping install keeps the old tag; completed install is picked up at the
next rollout start; strictly increasing; busy), written from the paper's text.
"""
from __future__ import annotations


class Busy(Exception):
    pass


class BadVersion(Exception):
    pass


class NoPolicy(Exception):
    pass


class WorkerVersions:
    def __init__(self, n_buffers: int = 2):
        self.n_buffers = n_buffers
        self.active = None          # version being served
        self.pending = None         # version being installed
        self.pending_done = False
        self.newest = None

    def offer(self, version: int):
        """A new snapshot starts installing."""
        if self.newest is not None and version <= self.newest:
            raise BadVersion(version)
        if self.pending is not None:
            raise Busy(version)
        if self.n_buffers == 1 or self.active is None:
            # single buffer, or nothing served yet: the install is the only policy
            self.active = None if self.n_buffers == 1 else self.active
        self.pending = version
        self.pending_done = False
        self.newest = version

    def install_complete(self):
        self.pending_done = True

    def begin_rollout(self) -> int:
        """Version that tags every trajectory of the rollout that starts now."""
        if self.pending is not None and (self.pending_done or self.active is None):
            # with nothing else to serve the worker waits for the install
            self.active, self.pending, self.pending_done = self.pending, None, False
        if self.active is None:
            raise NoPolicy()
        return self.active
