"""Host model of the barrier protocol of the fused score kernel: threads stand for the warp roles
of every CTA of one cluster, Python objects for the mbarriers.

What is modelled (names as in the kernel): per CTA a copy role (TMA), an MMA role, TWO exp roles
(the two groups of exp warps alternate heads: group g takes the heads g, g + 2, ...) and an add
role, joined by the barriers
    full / empty      staged keys of a head have landed / have been consumed        (n_q stages)
    tfull             logits of a head are in a tensor-memory buffer                 (n_buf buffers)
    eready            the exponentials of a head are in the buffer
    tempty            the buffer is free again
    sfull             every CTA's (max, sum) pair of a head has arrived in a slot    (n_slot slots)
with the phase-parity waits, the transaction counts of the asynchronous statistics stores, the
hand-over (an exp group hands a head's exponentials to the add role at once; ``handover="late"``
models the alternative - only when the group has got to its NEXT head, two heads on - which ends
in time-outs with two buffers: that next head needs the very same buffer), the
"tight" rule (the exp role stays within d heads of the local add role when there are only 2 d
slots) and the bounded waits: a wait that runs out raises the CTA's abort flag, every other wait
of that CTA then returns at once, the CTA records a time-out, tells its peers before the exit
barrier of the cluster, and the request is marked invalid (kept_cnt = -1).

Grid plans (``grid=True``): the CTAs of the request are no cluster; the exp role leaves its pair in
the CTA's own memory and arrives on ``gsent``; a publishing role stores the pair to (modelled)
global memory and adds one to the head's counter; a fetch role waits until the counter shows every
CTA, copies the head's pairs into a statistics slot and completes the slot's barrier - it learns
that a slot is free from the buffer barrier (``tempty``) of the head that used it, by parity.

The model checks what the kernel relies on: no statistics slot is written before its previous
content has been read, no buffer is refilled before it was released, every head is processed
exactly once per CTA, and a missing arrive ends in a clean time-out everywhere instead of a hang.
"""
import threading
import time

OK, TIMEOUT = 0, 6          # MUSTDROP_OK, MUSTDROP_ERR_TIMEOUT
N_GROUPS = 2                # groups of exp warps per CTA; they alternate heads


class ProtocolError(AssertionError):
    pass


class Mbarrier:
    """An mbarrier with an arrival count and a transaction count; a phase completes when both
    reach zero.  Transactions may be counted before the phase's expectation is armed."""

    def __init__(self, count):
        self.count = count
        self.pending = count
        self.tx = 0
        self.phase = 0
        self.lock = threading.Lock()

    def _maybe_complete(self):
        if self.pending == 0 and self.tx == 0:
            self.phase ^= 1
            self.pending = self.count

    def arrive(self, expect_tx=0):
        with self.lock:
            self.tx += expect_tx
            self.pending -= 1
            if self.pending < 0:
                raise ProtocolError("more arrivals than the barrier was initialised for")
            self._maybe_complete()

    def complete_tx(self, n):
        with self.lock:
            self.tx -= n
            self._maybe_complete()

    def try_wait(self, parity):
        with self.lock:
            return self.phase != parity     # the phase with this parity has completed


class Cta:
    def __init__(self, cluster, rank, geo):
        self.cluster, self.rank, self.geo = cluster, rank, geo
        self.abort = False
        self.status = OK
        self.full = [Mbarrier(1) for _ in range(geo["n_q"])]
        self.empty = [Mbarrier(1) for _ in range(geo["n_q"])]
        self.tfull = [Mbarrier(1) for _ in range(geo["n_buf"])]
        self.eready = [Mbarrier(1) for _ in range(geo["n_buf"])]
        self.tempty = [Mbarrier(1) for _ in range(geo["n_buf"])]
        self.sfull = [Mbarrier(1) for _ in range(geo["n_slot"])]
        self.gsent = [Mbarrier(1) for _ in range(geo["n_buf"])]     # grid plans: exp role -> publishing role
        self.own_pair = [None] * geo["n_buf"]
        self.stats = [[None] * geo["C"] for _ in range(geo["n_slot"])]   # head whose pair sits there
        self.stage_head = [None] * geo["n_q"]
        self.buf_state = [("free", None)] * geo["n_buf"]
        self.added = []                     # heads the add role finished, in order
        self.guard = threading.Lock()

    def wait(self, bar, parity, limit):
        """Bounded wait: False when it ran out or the CTA has already given up."""
        t0 = time.monotonic()
        while not bar.try_wait(parity):
            if self.abort or time.monotonic() - t0 > limit:
                self.abort = True
                return False
            time.sleep(0.0002)
        return True


class Cluster:
    """One request: C CTAs x 4 roles.  fault = (rank, role, head, what) makes that role skip one
    arrive ("full", "tfull", "eready", "tempty", "empty") or one statistics store ("stats")."""

    def __init__(self, C=2, H=12, n_q=2, n_buf=3, n_slot=None, tight=0, limit=0.25, fault=None, jitter=None,
                 grid=False, handover="auto"):
        n_slot = (min(n_buf, 4) if grid else 2 * n_buf) if n_slot is None else n_slot
        self.grid = grid
        self.g_lock = threading.Lock()
        self.g_cnt = [0] * H                       # global memory: pairs published per head
        self.g_pairs = [[None] * C for _ in range(H)]
        self.geo = dict(C=C, H=H, n_q=n_q, n_buf=n_buf, n_slot=n_slot, tight=tight)
        # "auto": what the kernel does (at once); "late": one head of the group later
        self.eager = handover == "auto"
        self.limit, self.fault, self.jitter = limit, fault, jitter or {}
        self.ctas = [Cta(self, r, self.geo) for r in range(C)]
        self.errors = []
        self.cluster_abort = False
        self.kept_cnt = None

    def _skips(self, rank, role, h, what):
        return self.fault == (rank, role, h, what)

    def _pause(self, rank, role):
        d = self.jitter.get((rank, role), 0.0)
        if d:
            time.sleep(d)

    # ---- the roles ---------------------------------------------------------------------------------
    def tma(self, c):
        g = self.geo
        for h in range(g["H"]):
            s = h % g["n_q"]
            if not c.wait(c.empty[s], ((h // g["n_q"]) & 1) ^ 1, self.limit):
                return
            self._pause(c.rank, "tma")
            if c.stage_head[s] is not None:
                raise ProtocolError("stage %d refilled before head %s was consumed" % (s, c.stage_head[s]))
            c.stage_head[s] = h
            if not self._skips(c.rank, "tma", h, "full"):
                c.full[s].arrive()

    def mma(self, c):
        g = self.geo
        for h in range(g["H"]):
            s, buf = h % g["n_q"], h % g["n_buf"]
            if not c.wait(c.full[s], (h // g["n_q"]) & 1, self.limit):
                return
            if not c.wait(c.tempty[buf], ((h // g["n_buf"]) & 1) ^ 1, self.limit):
                return
            self._pause(c.rank, "mma")
            if c.stage_head[s] != h:
                raise ProtocolError("MMA of head %d found head %s staged" % (h, c.stage_head[s]))
            with c.guard:
                if c.buf_state[buf][0] != "free":
                    raise ProtocolError("buffer %d overwritten while %s" % (buf, c.buf_state[buf],))
                c.buf_state[buf] = ("logits", h)
            c.stage_head[s] = None
            if not self._skips(c.rank, "mma", h, "empty"):
                c.empty[s].arrive()
            if self._skips(c.rank, "mma", h, "tfull"):
                return      # MMAs complete in order: if this head's never do, no later commit arrives either
            c.tfull[buf].arrive()

    def exp(self, c, grp=0):
        g = self.geo
        last = None                                   # head this group worked on before, not yet handed over
        for h in range(grp, g["H"], N_GROUPS):
            buf, slot = h % g["n_buf"], h % g["n_slot"]
            if g["tight"] and h >= g["tight"]:
                u = h - g["tight"]
                if not c.wait(c.tempty[u % g["n_buf"]], (u // g["n_buf"]) & 1, self.limit):
                    return
            if not c.wait(c.tfull[buf], (h // g["n_buf"]) & 1, self.limit):
                return
            if not self.grid:
                c.sfull[slot].arrive(expect_tx=g["C"])    # arm: every CTA will send one pair
            if last is not None:                          # late hand-over of the group's previous head
                if not self._skips(c.rank, "exp", last, "eready"):
                    c.eready[last % g["n_buf"]].arrive()
                last = None
            self._pause(c.rank, "exp")
            with c.guard:
                if c.buf_state[buf] != ("logits", h):
                    raise ProtocolError("exp role of head %d found %s" % (h, c.buf_state[buf],))
                c.buf_state[buf] = ("exps", h)
            if self.grid:
                if c.own_pair[buf] is not None:
                    raise ProtocolError("own pair of buffer %d overwritten before head %s was added" % (buf, c.own_pair[buf]))
                c.own_pair[buf] = h
                if not self._skips(c.rank, "exp", h, "stats"):
                    c.gsent[buf].arrive()
            elif not self._skips(c.rank, "exp", h, "stats"):
                for peer in self.ctas:                    # st.async into every CTA, counted on ITS barrier
                    with peer.guard:
                        if peer.stats[slot][c.rank] is not None:
                            raise ProtocolError("slot %d of CTA %d overwritten: head %s unread, head %d arrives"
                                                % (slot, peer.rank, peer.stats[slot][c.rank], h))
                        peer.stats[slot][c.rank] = h
                    peer.sfull[slot].complete_tx(1)
            if self.eager:
                if not self._skips(c.rank, "exp", h, "eready"):
                    c.eready[buf].arrive()
            else:
                last = h
        if last is not None and not self._skips(c.rank, "exp", last, "eready"):
            c.eready[last % g["n_buf"]].arrive()          # the last head the group worked on

    def exp1(self, c):
        self.exp(c, 1)

    def add(self, c):
        g = self.geo
        for h in range(g["H"]):
            buf, slot = h % g["n_buf"], h % g["n_slot"]
            if not c.wait(c.sfull[slot], (h // g["n_slot"]) & 1, self.limit):
                return
            with c.guard:
                if c.stats[slot] != [h] * g["C"]:
                    raise ProtocolError("add role of head %d read pairs of heads %s" % (h, c.stats[slot]))
                c.stats[slot] = [None] * g["C"]
                if self.grid:
                    if c.own_pair[buf] != h:
                        raise ProtocolError("add role of head %d found own pair of head %s" % (h, c.own_pair[buf]))
                    c.own_pair[buf] = None
            if not c.wait(c.eready[buf], (h // g["n_buf"]) & 1, self.limit):
                return
            self._pause(c.rank, "add")
            with c.guard:
                if c.buf_state[buf] != ("exps", h):
                    raise ProtocolError("add role of head %d found %s" % (h, c.buf_state[buf],))
                c.buf_state[buf] = ("free", None)
            c.added.append(h)
            if not self._skips(c.rank, "add", h, "tempty"):
                c.tempty[buf].arrive()

    def publish(self, c):
        g = self.geo
        for h in range(g["H"]):
            buf = h % g["n_buf"]
            if not c.wait(c.gsent[buf], (h // g["n_buf"]) & 1, self.limit):
                return
            self._pause(c.rank, "publish")
            with self.g_lock:
                self.g_pairs[h][c.rank] = h
                if not self._skips(c.rank, "publish", h, "count"):
                    self.g_cnt[h] += 1

    def fetch(self, c):
        g = self.geo
        for h in range(g["H"]):
            slot = h % g["n_slot"]
            self._pause(c.rank, "fetch_late")       # (a fetch role that gets to its next head late)
            if h >= g["n_slot"]:
                u = h - g["n_slot"]
                if not c.wait(c.tempty[u % g["n_buf"]], (u // g["n_buf"]) & 1, self.limit):
                    return
            t0 = time.monotonic()
            while True:
                with self.g_lock:
                    if self.g_cnt[h] >= g["C"]:
                        break
                if c.abort or time.monotonic() - t0 > self.limit:
                    c.abort = True
                    return
                time.sleep(0.0002)
            self._pause(c.rank, "fetch")
            with c.guard:
                if c.stats[slot] != [None] * g["C"]:
                    raise ProtocolError("slot %d of CTA %d refilled for head %d before heads %s were read"
                                        % (slot, c.rank, h, c.stats[slot]))
                c.stats[slot] = list(self.g_pairs[h])
            c.sfull[slot].arrive()

    # ---- a run ---------------------------------------------------------------------------------------
    def run(self, join_limit=20.0):
        """Run all roles to their common exit.  Returns True when every thread came back."""
        def guarded(fn, c):
            try:
                fn(c)
            except ProtocolError as e:          # a broken invariant: remember it, let the others time out
                self.errors.append(str(e))
                c.abort = True

        roles = (self.tma, self.mma, self.exp, self.exp1, self.add) + ((self.publish, self.fetch) if self.grid else ())
        threads = [threading.Thread(target=guarded, args=(fn, c), daemon=True)
                   for c in self.ctas for fn in roles]
        for t in threads:
            t.start()
        t_end = time.monotonic() + join_limit
        for t in threads:
            t.join(max(0.0, t_end - time.monotonic()))
        if any(t.is_alive() for t in threads):
            return False
        # the common exit: each CTA records its own time-out and tells its peers, cluster barrier,
        # then rank 0 marks the request invalid if anyone gave up
        for c in self.ctas:
            if c.abort:
                c.status = TIMEOUT
                self.cluster_abort = True
        self.kept_cnt = -1 if self.cluster_abort else self.geo["H"]
        return True
