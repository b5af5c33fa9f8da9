"""The barrier protocol of the fused score kernel on a host model (threads as warp roles, one
cluster): it completes for the geometries the planner produces, its slot and buffer counts are
exactly enough, and a role that skips an arrive ends in a time-out in every CTA - no hang."""
import pytest

from protocol_model import OK, TIMEOUT, Cluster

GEOMETRIES = [
    dict(C=1, n_q=2, n_buf=3),
    dict(C=2, n_q=2, n_buf=3),                       # the 7B batch-64 plan
    dict(C=4, n_q=4, n_buf=6),
    dict(C=5, n_q=2, n_buf=3),
    dict(C=4, n_q=2, n_buf=2),                       # 176-column tiles: two buffers only
    dict(C=8, n_q=3, n_buf=8),
    dict(C=10, n_q=2, n_buf=3, n_slot=4, tight=2),   # large clusters: few slots, the exp role held near the add role
    dict(C=12, n_q=2, n_buf=3, n_slot=2, tight=1),
]


@pytest.mark.parametrize("geo", GEOMETRIES, ids=lambda g: "C%d_q%d_b%d_s%s" % (g["C"], g["n_q"], g["n_buf"], g.get("n_slot", "2b")))
def test_protocol_completes_and_keeps_its_invariants(geo):
    cl = Cluster(H=13, limit=5.0, **geo)
    assert cl.run(), "a role never came back"
    assert cl.errors == []
    for c in cl.ctas:
        assert c.status == OK and c.added == list(range(13))
    assert cl.kept_cnt == 13


@pytest.mark.parametrize("slow", [(0, "add"), (1, "exp"), (0, "tma"), (1, "mma")])
def test_protocol_tolerates_a_slow_role(slow):
    # one role of one CTA is much slower than its peers: they run ahead as far as the barriers allow
    cl = Cluster(C=3, H=10, n_q=2, n_buf=3, limit=5.0, jitter={slow: 0.01})
    assert cl.run() and cl.errors == []
    assert all(c.added == list(range(10)) for c in cl.ctas) and cl.kept_cnt == 10


@pytest.mark.parametrize("n_buf,ends", [(2, False), (3, True), (4, True)])
def test_a_late_hand_over_needs_a_third_buffer(n_buf, ends):
    # Had an exp group handed a head over only when it has got to its next head, two heads on:
    # with two buffers that next head needs the same buffer - its MMAs wait for the add role, which
    # waits for the hand-over - and every wait runs out.  (The kernel hands over at once.)
    cl = Cluster(C=2, H=9, n_q=2, n_buf=n_buf, limit=0.3, handover="late")
    assert cl.run(join_limit=10.0), "a role hung instead of giving up"
    assert cl.errors == []
    assert (cl.kept_cnt == 9) == ends
    if not ends:
        assert all(c.status == TIMEOUT for c in cl.ctas)


def test_fewer_slots_than_the_protocol_needs_is_caught_by_the_model():
    # 2 x buffers slots are needed without the tight rule: with fewer, a fast peer overwrites an unread pair
    cl = Cluster(C=2, H=16, n_q=4, n_buf=4, n_slot=4, tight=0, limit=0.3, jitter={(0, "add"): 0.01})
    cl.run()
    assert cl.errors and cl.cluster_abort and cl.kept_cnt == -1


FAULTS = [
    (1, "tma", 3, "full"),      # a copy that never completes
    (0, "mma", 2, "tfull"),     # the MMA role does not hand the logits over
    (1, "mma", 4, "empty"),     # a stage is never released
    (0, "exp", 5, "eready"),    # the exponentials are never handed over
    (1, "exp", 1, "stats"),     # one CTA's statistics never arrive anywhere
    (0, "add", 3, "tempty"),    # a buffer is never freed
]


@pytest.mark.parametrize("tight", [0, 2])
@pytest.mark.parametrize("fault", FAULTS, ids=lambda f: "cta%d_%s_h%d_%s" % f)
def test_a_skipped_arrive_times_out_everywhere(fault, tight):
    geo = dict(C=3, n_q=2, n_buf=3, n_slot=4, tight=2) if tight else dict(C=2, n_q=2, n_buf=3)
    cl = Cluster(H=12, limit=0.2, fault=fault, **geo)
    assert cl.run(join_limit=10.0), "a role hung instead of giving up"
    assert cl.errors == []                                   # the invariants held up to the give-up
    assert all(c.status == TIMEOUT for c in cl.ctas)         # every CTA of the cluster reports the time-out
    assert cl.cluster_abort and cl.kept_cnt == -1            # and the request is marked invalid
    assert all(len(c.added) < 12 for c in cl.ctas)


# ---- grid plans: statistics through (modelled) global memory, publishing and fetch roles -----------

GRID_GEOMETRIES = [
    dict(C=2, n_q=2, n_buf=3),                # slots default to min(buffers, 4)
    dict(C=6, n_q=3, n_buf=5, n_slot=3),
    dict(C=17, n_q=2, n_buf=4, n_slot=4),     # the video workload's plan
    dict(C=5, n_q=4, n_buf=8, n_slot=6),
]


@pytest.mark.parametrize("geo", GRID_GEOMETRIES, ids=lambda g: "C%d_b%d_s%s" % (g["C"], g["n_buf"], g.get("n_slot", "d")))
def test_grid_protocol_completes_and_keeps_its_invariants(geo):
    cl = Cluster(H=13, limit=5.0, grid=True, **geo)
    assert cl.run(), "a role never came back"
    assert cl.errors == []
    for c in cl.ctas:
        assert c.status == OK and c.added == list(range(13))


@pytest.mark.parametrize("slow", [(0, "fetch"), (0, "fetch_late"), (1, "publish"), (0, "add"), (1, "exp")])
def test_grid_protocol_tolerates_a_slow_role(slow):
    cl = Cluster(C=3, H=10, n_q=2, n_buf=3, limit=5.0, grid=True, jitter={slow: 0.01})
    assert cl.run() and cl.errors == []
    assert all(c.added == list(range(10)) for c in cl.ctas)


def test_more_slots_than_buffers_stalls_the_fetch_role():
    # the fetch role reads "slot free" off the parity of a buffer barrier: with four slots on three
    # buffers the add role can finish a second head on that buffer before a slow fetch role looks,
    # the parity is back where it was, and the wait runs out (seen once on the GPU: 0.1 s per call).
    # With no more slots than buffers the same slow role is harmless (test above).
    cl = Cluster(C=2, H=16, n_q=2, n_buf=3, n_slot=4, limit=0.3, grid=True, jitter={(0, "fetch_late"): 0.02})
    assert cl.run(join_limit=15.0), "a role hung instead of giving up"
    assert cl.cluster_abort and cl.kept_cnt == -1


@pytest.mark.parametrize("fault", [(1, "publish", 3, "count"), (0, "exp", 2, "stats"), (1, "add", 4, "tempty")],
                         ids=lambda f: "cta%d_%s_h%d_%s" % f)
def test_grid_protocol_times_out_everywhere_after_a_skipped_signal(fault):
    cl = Cluster(C=3, H=12, n_q=2, n_buf=3, limit=0.2, fault=fault, grid=True)
    assert cl.run(join_limit=10.0), "a role hung instead of giving up"
    assert cl.errors == []
    assert all(c.status == TIMEOUT for c in cl.ctas)
    assert cl.kept_cnt == -1
