"""A copy engine for host-side tests of the expert store: no GPU, plain host memory, and an
adversarial scheduler.  Every operation the store issues (copy, fill, event record, stream wait) is
only queued on its stream; nothing happens until the scheduler runs, and then it picks, at random,
any stream whose next operation is allowed to run.  Operations of one stream keep their order; across
streams the only orderings are the ones the store asked for with events.  A copy therefore lands
late, and in any interleaving with the other stream that the store's events permit -- if the store
forgets an ordering it needs, some schedule shows it.

The test plays the compute side: it queues `kernel` operations (Python callables) on a compute
stream; they run when the scheduler reaches them and check what a kernel would read.
"""
import ctypes as C
import random


class FakeEngine:
    def __init__(self, seed=0):
        self.rng = random.Random(seed)
        self.queues = {}                  # stream id -> list of pending ops
        self.next_event = 1
        self.tokens = {}                  # event id -> latest record token (a one-element list: [done?])
        self.allocs = {}
        self.log = []                     # executed ops, in execution order
        self.copies_done = 0

    # ---- the ten entry points (ctx is dropped by the binding)
    def copy_h2d(self, ctx, dst, src, n, stream):
        self._q(stream).append(("copy", dst, src, n))
        return 0

    def fill(self, ctx, dst, byte, n, stream):
        self._q(stream).append(("fill", dst, byte, n))
        return 0

    def event_create(self, ctx, out):
        out[0] = self.next_event
        self.tokens[self.next_event] = None
        self.next_event += 1
        return 0

    def event_destroy(self, ctx, ev):
        self.tokens.pop(ev, None)
        return 0

    def event_record(self, ctx, ev, stream):
        tok = [False]
        self.tokens[ev] = tok
        self._q(stream).append(("record", tok))
        return 0

    def stream_wait_event(self, ctx, stream, ev):
        tok = self.tokens.get(ev)
        if tok is not None:               # waiting on an event never recorded is a no-op
            self._q(stream).append(("wait", tok))
        return 0

    def event_synchronize(self, ctx, ev):
        tok = self.tokens.get(ev)
        while tok is not None and not tok[0]:
            if not self.step():
                return -5                 # deadlock: nothing can run
        return 0

    def stream_synchronize(self, ctx, stream):
        while self._q(stream):
            if not self.step():
                return -5
        return 0

    def host_alloc(self, ctx, out, n):
        buf = C.create_string_buffer(n)
        out[0] = C.addressof(buf)
        self.allocs[C.addressof(buf)] = buf
        return 0

    def host_free(self, ctx, ptr):
        self.allocs.pop(ptr, None)
        return 0

    # ---- the test's side
    def kernel(self, stream, fn):
        """Queues a callable on a stream: the stand-in for a kernel launch."""
        self._q(stream).append(("kernel", fn))

    def _q(self, stream):
        return self.queues.setdefault(stream or 0, [])

    def _runnable(self):
        out = []
        for sid, q in self.queues.items():
            if q and (q[0][0] != "wait" or q[0][1][0]):
                out.append(sid)
        return out

    def step(self):
        """Runs one operation of a randomly chosen runnable stream; False if none can run."""
        ready = self._runnable()
        if not ready:
            return False
        sid = self.rng.choice(ready)
        op = self.queues[sid].pop(0)
        kind = op[0]
        if kind == "copy":
            C.memmove(op[1], op[2], op[3])
            self.copies_done += 1
        elif kind == "fill":
            C.memset(op[1], op[2], op[3])
        elif kind == "record":
            op[1][0] = True
        elif kind == "kernel":
            op[1]()
        self.log.append((sid, kind))
        return True

    def run_some(self, n):
        for _ in range(n):
            if not self.step():
                break

    def drain(self):
        while self.step():
            pass
        return all(not q for q in self.queues.values())
