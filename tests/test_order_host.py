"""The host-side rules that order decode calls issued on one stream, checked through the
library's host-only model of them (no device): every hazard between two calls in flight
together must be covered by what the later call waits for, and nothing else may serialise."""
import random

import pytest

IO = 64 * 1024      # bytes of q / out
KV = 16 * 1024      # bytes of k_new / v_new
WS = 0x7000_0000_0000
NEED = 1 << 20


@pytest.fixture()
def zc():
    from paper_2405_14256_b200 import build
    build.build()
    import paper_2405_14256_b200 as mod
    mod.load_library()
    mod.zc_order_model_reset()
    return mod


def call(zc, stream=1, cache=0, q=0x1000_0000, k=0, v=0, out=0x2000_0000, collect=False,
         ws=WS, ws_bytes=16 * NEED, need=NEED, capture=0):
    return zc.zc_order_model_call(stream, cache, q, k, v, out, IO, KV, collect, ws, ws_bytes, need, capture)


def test_first_call_opens_an_epoch_and_later_calls_join_it(zc):
    r0 = call(zc, q=0x1000_0000, out=0x2000_0000)
    assert r0["epoch_start"] == 1 and r0["e"] == 0 and r0["slot"] == 0
    for i in range(1, 40):
        r = call(zc, q=0x1000_0000 + i * IO, out=0x2000_0000 + i * IO)
        assert r["epoch_start"] == 0 and r["e"] == i and r["tag"] == r0["tag"]
        assert r["slot"] == i % 16
        # independent buffers: only the workspace region (16 of them) is waited for
        assert r["need_start"] <= 0
        assert r["need_end"] == i - 16 + 1


def test_workspace_regions_and_counters_bound_the_calls_in_flight(zc):
    for regions in (1, 2, 5, 64, 200):
        zc.zc_order_model_reset()
        k = min(64, regions)
        for i in range(3 * k + 2):
            r = call(zc, q=0x1000_0000 + i * IO, out=0x2000_0000 + i * IO, ws_bytes=regions * NEED)
            assert r["slot"] == i % k
            assert r["need_end"] == i - k + 1      # call i - k used the same region
            assert r["need_start"] <= max(0, i - 63)


def test_read_after_write_waits_before_the_inputs_are_read(zc):
    call(zc, q=0x1000_0000, out=0x2000_0000)
    call(zc, q=0x1100_0000, out=0x2100_0000)
    r = call(zc, q=0x2000_0000, out=0x2200_0000)           # reads call 0's output
    assert r["need_start"] == 1
    r = call(zc, q=0x2100_0000 + IO - 2, out=0x2300_0000)  # overlaps call 1's output by 2 bytes
    assert r["need_start"] == 2
    r = call(zc, q=0x2100_0000 + IO, out=0x2400_0000)      # adjacent, not overlapping
    assert r["need_start"] <= 0
    r = call(zc, q=0x1200_0000, k=0x2200_0000, v=0x3000_0000, out=0x2500_0000)   # k_new = call 2's output
    assert r["need_start"] == 3


def test_write_hazards_wait_before_anything_is_written(zc):
    call(zc, q=0x1000_0000, out=0x2000_0000)
    r = call(zc, q=0x1100_0000, out=0x2000_0000)           # same output buffer
    assert r["need_end"] == 1 and r["need_start"] <= 0
    r = call(zc, q=0x1200_0000, out=0x1100_0000)           # overwrites call 1's q
    assert r["need_end"] == 2
    call(zc, q=0x1300_0000, k=0x1400_0000, v=0x1500_0000, out=0x2300_0000)
    r = call(zc, cache=1, q=0x1600_0000, out=0x1500_0000 + KV - 1)   # overwrites the last byte of call 3's v_new
    assert r["need_end"] == 4
    r = call(zc, cache=1, q=0x1700_0000, out=0x1500_0000 - IO)       # ends where that v_new begins
    assert r["need_end"] <= 0


def test_probe_steps_of_one_cache_are_ordered_among_themselves(zc):
    call(zc, cache=0, q=0x1000_0000, out=0x2000_0000, collect=True)
    r = call(zc, cache=1, q=0x1100_0000, out=0x2100_0000, collect=True)
    assert r["need_end"] <= 0                               # another cache's statistics
    r = call(zc, cache=0, q=0x1200_0000, out=0x2200_0000, collect=False)
    assert r["need_end"] <= 0                               # adds nothing
    r = call(zc, cache=0, q=0x1300_0000, out=0x2300_0000, collect=True)
    assert r["need_end"] == 1
    r = call(zc, cache=1, q=0x1400_0000, out=0x2400_0000, collect=True)
    assert r["need_end"] == 2


def test_a_stored_tail_row_is_complete_before_the_caches_next_call_reads_it(zc):
    call(zc, cache=0, q=0x1000_0000, k=0x3000_0000, v=0x3100_0000, out=0x2000_0000)
    r = call(zc, cache=1, q=0x1100_0000, k=0x3200_0000, v=0x3300_0000, out=0x2100_0000)
    assert r["need_start"] <= 0
    r = call(zc, cache=0, q=0x1200_0000, k=0x3400_0000, v=0x3500_0000, out=0x2200_0000)
    assert r["need_start"] == 1                             # call 0 stored cache 0's previous row
    r = call(zc, cache=1, q=0x1300_0000, out=0x2300_0000)
    assert r["need_start"] == 2
    r = call(zc, cache=1, q=0x1400_0000, out=0x2400_0000)   # call 3 stored nothing
    assert r["need_start"] == 2


def test_a_change_in_an_earlier_epoch_needs_no_wait(zc):
    call(zc, cache=2, q=0x1000_0000, k=0x3000_0000, v=0x3100_0000, out=0x2000_0000)
    call(zc, cache=3, q=0x1300_0000, out=0x2300_0000, ws_bytes=8 * NEED)   # new workspace: new epoch
    r = call(zc, cache=2, q=0x1400_0000, out=0x2400_0000, ws_bytes=8 * NEED)
    assert r["e"] == 1 and r["need_start"] <= 0              # that kernel completed before the epoch began


def test_epoch_restarts(zc):
    r = call(zc)
    tag = r["tag"]
    r = call(zc, q=0x1100_0000, out=0x2100_0000)
    assert r["epoch_start"] == 0
    r = call(zc, q=0x1200_0000, out=0x2200_0000, ws=WS + 4096)          # another workspace
    assert r["epoch_start"] == 1 and r["e"] == 0 and r["tag"] == (tag + 1) & 0xFFF
    r = call(zc, q=0x1300_0000, out=0x2300_0000, ws=WS + 4096, need=2 * NEED)   # does not fit a region
    assert r["epoch_start"] == 1 and r["tag"] == (tag + 2) & 0xFFF
    r = call(zc, q=0x1400_0000, out=0x2400_0000, ws=WS + 4096, need=NEED)       # a smaller call joins
    assert r["epoch_start"] == 0 and r["slot"] == 1
    r = call(zc, q=0x1500_0000, out=0x2500_0000, ws=WS + 4096, capture=7)       # stream capture begins
    assert r["epoch_start"] == 1
    r = call(zc, q=0x1600_0000, out=0x2600_0000, ws=WS + 4096, capture=7)
    assert r["epoch_start"] == 0
    r = call(zc, q=0x1700_0000, out=0x2700_0000, ws=WS + 4096, capture=8)       # another capture
    assert r["epoch_start"] == 1
    r = call(zc, q=0x1800_0000, out=0x2800_0000, ws=WS + 4096)                  # capture ended
    assert r["epoch_start"] == 1


def test_streams_have_records_of_their_own_and_the_oldest_is_recycled(zc):
    recs = {}
    for s in range(1, 17):
        r = call(zc, stream=s)
        assert r["epoch_start"] == 1 and r["drain"] == 0
        recs[s] = r["record"]
    assert sorted(recs.values()) == list(range(16))
    r = call(zc, stream=5, q=0x1100_0000, out=0x2100_0000)
    assert r["record"] == recs[5] and r["epoch_start"] == 0 and r["e"] == 1
    call(zc, stream=1, q=0x1100_0000, out=0x2100_0000)       # stream 2 is now the least recently used
    r = call(zc, stream=99)
    assert r["record"] == recs[2] and r["drain"] == 1 and r["epoch_start"] == 1
    r = call(zc, stream=2)                                   # comes back on another record, as a new epoch
    assert r["epoch_start"] == 1 and r["drain"] == 1 and r["record"] == recs[3]


def test_epoch_ends_before_the_call_index_outgrows_its_field(zc):
    tag = call(zc)["tag"]
    last = None
    n = (1 << 20) - 1
    for i in range(1, n + 2):
        r = call(zc, q=0x1000_0000 + (i % 7) * IO, out=0x2000_0000 + (i % 64) * IO)
        if r["epoch_start"]:
            last = (i, r)
            break
        assert r["e"] == i and r["e"] < (1 << 20)
    assert last is not None and last[0] == n
    assert last[1]["e"] == 0 and last[1]["tag"] == (tag + 1) & 0xFFF


def test_tag_wraps_at_twelve_bits(zc):
    tags = [call(zc, ws=WS + 256 * i)["tag"] for i in range(5000)]
    assert all(0 <= t < 4096 for t in tags)
    assert all(tags[i + 1] == (tags[i] + 1) & 0xFFF for i in range(len(tags) - 1))


def test_random_schedules_cover_every_hazard(zc):
    """Brute force: replay random calls over a small pool of buffers and caches and check, for
    every pair of calls of an epoch, that a hazard between them implies the wait."""
    rng = random.Random(1234)
    bufs = [0x1000_0000 + i * IO for i in range(12)]
    kvbufs = [0x4000_0000 + i * KV for i in range(6)]
    for trial in range(20):
        zc.zc_order_model_reset()
        regions = rng.choice([1, 3, 16, 64, 100])
        log = []
        for i in range(300):
            q, out = rng.sample(bufs, 2)
            store = rng.random() < 0.5
            k, v = (rng.sample(kvbufs, 2) if store else (0, 0))
            if rng.random() < 0.1:
                k = rng.choice(bufs)            # a k_new that aliases some q / out buffer
                v = v or kvbufs[0]
            cache = rng.randrange(3)
            collect = rng.random() < 0.3
            r = call(zc, cache=cache, q=q, k=k, v=v, out=out, collect=collect, ws_bytes=regions * NEED)
            assert r["e"] == i
            me = dict(q=q, k=k, v=v, out=out, cache=cache, collect=collect, store=bool(k), r=r)
            ins = [(q, IO)] + ([(k, KV), (v, KV)] if k else [])
            hit = lambda a, b: a[0] < b[0] + b[1] and b[0] < a[0] + a[1]
            for j, o in enumerate(log):
                o_ins = [(o["q"], IO)] + ([(o["k"], KV), (o["v"], KV)] if o["k"] else [])
                raw = any(hit(x, (o["out"], IO)) for x in ins)
                tail = o["store"] and o["cache"] == cache
                if raw or tail:
                    assert r["need_start"] >= j + 1, (trial, i, j)
                war = any(hit((out, IO), x) for x in o_ins)
                waw = hit((out, IO), (o["out"], IO))
                stats = collect and o["collect"] and o["cache"] == cache
                region = (i - j) % min(64, regions) == 0
                if war or waw or stats or region:
                    assert r["need_end"] >= j + 1, (trial, i, j)
            assert r["need_start"] <= i and r["need_end"] <= i
            log.append(me)
