"""Property tests (hypothesis) of the host-side table builders: whatever the tensor
sizes, alignment phases, chunk lengths, row counts and world sizes, every element /
row is covered exactly once and the documented bounds hold."""
import numpy as np
from hypothesis import given, settings
from hypothesis import strategies as st

from paper_2601_07876_b200 import binding as B
from paper_2601_07876_b200 import sharding

sizes = st.lists(st.integers(min_value=1, max_value=40_000), min_size=1, max_size=12)


@settings(max_examples=60, deadline=None)
@given(numel=sizes, data=st.data())
def test_chunk_table_covers_every_element_once(numel, data):
    phase = [data.draw(st.integers(0, 31)) for _ in numel]
    chunk = data.draw(st.sampled_from([1024, 2048, 4096, 8192]))
    t, off, ln = B.novak_build_chunks(numel, phase, chunk)
    seen = [np.zeros(n, dtype=np.int8) for n in numel]
    last = (-1, 0)
    for ti, oi, li in zip(t, off, ln):
        assert 0 < li <= chunk
        assert (ti, oi) > last                      # tensor order, then element order
        last = (ti, oi)
        seen[ti][oi:oi + li] += 1
        if oi > 0:                                  # after the head entry: 128-byte aligned
            assert (phase[ti] + oi) % 32 == 0
    assert all((s == 1).all() for s in seen)


@settings(max_examples=60, deadline=None)
@given(data=st.data())
def test_row_units_cover_every_row_once(data):
    n = data.draw(st.integers(1, 8))
    numel, rows = [], []
    for _ in range(n):
        if data.draw(st.booleans()):
            r = data.draw(st.integers(1, 600))
            length = data.draw(st.sampled_from([1, 2, 3, 5, 27, 64, 127, 128, 129, 576, 1024, 2048,
                                                2049, 4608, 8192, 8193, 16384, 16385, 40_000]))
            numel.append(r * length)
            rows.append(r)
        else:
            numel.append(data.draw(st.integers(1, 5000)))
            rows.append(0)
    units = B.novak_build_row_units(numel, rows)
    seen = {i: np.zeros((r, numel[i] // r), dtype=np.int8) for i, r in enumerate(rows) if r}
    for t, row0, n_rows, part_off, part_len in units:
        L = numel[t] // rows[t]
        if part_len:
            assert L > 8192 and n_rows == 1 and part_len <= 16384
            seen[t][row0, part_off:part_off + part_len] += 1
        else:
            assert L <= 8192
            seen[t][row0:row0 + n_rows] += 1
    assert all((s == 1).all() for s in seen.values())
    assert {u[0] for u in units} == set(seen)


@settings(max_examples=60, deadline=None)
@given(data=st.data())
def test_own_units_cover_the_rows_of_owned_tensors_once(data):
    """Units of the step kernel that forms its row means itself: every row of every tensor
    whose rows have at most 32768 elements exactly once, whole rows only, at most 256 rows
    and (beyond one row) at most 4096 elements per unit; nothing for longer rows."""
    n = data.draw(st.integers(1, 8))
    numel, rows = [], []
    for _ in range(n):
        if data.draw(st.booleans()):
            r = data.draw(st.integers(1, 600))
            length = data.draw(st.sampled_from([1, 2, 3, 5, 15, 16, 17, 27, 64, 147, 576, 2048, 2049,
                                                4096, 4097, 4608, 32768, 32769, 40_000]))
            numel.append(r * length)
            rows.append(r)
        else:
            numel.append(data.draw(st.integers(1, 5000)))
            rows.append(0)
    units = B.novak_build_own_units(numel, rows)
    owned = {i for i, r in enumerate(rows) if r and numel[i] // r <= 32768}
    seen = {i: np.zeros(rows[i], dtype=np.int8) for i in owned}
    for t, row0, n_rows in units:
        assert t in owned and 1 <= n_rows <= 256
        L = numel[t] // rows[t]
        assert n_rows == 1 or n_rows * L <= 4096
        seen[t][row0:row0 + n_rows] += 1
    assert all((s == 1).all() for s in seen.values())
    # consecutive units of a tensor are adjacent and in order
    for (t0, r0, n0), (t1, r1, _) in zip(units, units[1:]):
        assert (t1 == t0 and r1 == r0 + n0) or (t1 > t0 and r1 == 0)


@settings(max_examples=80, deadline=None)
@given(counts=st.lists(st.integers(1, 40), min_size=1, max_size=30), lead=st.integers(0, 120),
       group=st.integers(1, 8))
def test_adapt_items_cover_the_table_and_the_lag_orders_statistics_before_updates(counts, lead, group):
    """Work list of the one-launch layer adaptation: every chunk-table entry in exactly one
    item, items in tensor order; an item is a run of at most `group` entries of one tensor,
    the tensor's first entry (the only one but its last that may be short) alone.  CTA b
    takes the statistics of item b and the update of item b - lag: every statistics part
    an update waits for belongs to a CTA with a lower index or to the CTA itself (what the
    kernel's freedom from deadlock rests on), and the lag is no shorter than the lead asks."""
    first = np.concatenate([[0], np.cumsum(counts)]).tolist()
    items, lag = B.novak_build_adapt_order(first, lead, group)
    total = first[-1]
    tensor_of = np.repeat(np.arange(len(counts)), counts)
    covered = []
    for c, k in items:
        assert 1 <= k <= group
        assert len(set(tensor_of[c:c + k])) == 1            # one tensor
        if c == first[tensor_of[c]]:
            assert k == 1                                       # its first entry stands alone
        covered.extend(range(c, c + k))
    assert covered == list(range(total))                       # once each, tensors in order
    item_tensor = [int(tensor_of[c]) for c, _ in items]
    last_item = {t: i for i, t in enumerate(item_tensor)}
    for u, t in enumerate(item_tensor):
        cta = u + lag                                           # the CTA that updates item u
        assert last_item[t] <= cta                              # statistics of the whole tensor: earlier CTAs or its own
    longest = max(np.bincount(item_tensor))
    assert lag == longest - 1 + -(-lead // group)


@settings(max_examples=60, deadline=None)
@given(numel=sizes, world=st.integers(1, 9), align=st.sampled_from([1, 4, 64]))
def test_rank_partition_covers_every_element_once_and_is_balanced(numel, world, align):
    parts = sharding.partition_flat(numel, world, align)
    assert len(parts) == world
    seen = [np.zeros(n, dtype=np.int8) for n in numel]
    counts = []
    for slices in parts:
        c = 0
        for t, a, b in slices:
            assert 0 <= a < b <= numel[t]
            seen[t][a:b] += 1
            c += b - a
        counts.append(c)
    assert all((s == 1).all() for s in seen)
    total = sum(numel)
    assert max(counts) - min(counts) <= max(2 * align, total - (total // align) * align + align)


@settings(max_examples=150, deadline=None)
@given(beta1=st.floats(0.0, 0.9999), beta2=st.floats(0.0, 0.99999),
       lr=st.floats(1e-6, 1.0), wd=st.floats(0.0, 1.0), k=st.integers(0, 12),
       t=st.one_of(st.integers(1, 200), st.integers(200, 10 ** 7)),
       adaptive=st.booleans(), rectified=st.booleans())
def test_planner_agrees_with_the_oracle_for_any_hyperparameters(beta1, beta2, lr, wd, k, t,
                                                                adaptive, rectified):
    """The library's host plan (double, -expm1(t log beta)) against the oracle's scalars
    (long double powers): Eq. 3-9, 18, the branch of Eq. 8 and the sync schedule.  Where
    rho_t comes within 1e-6 of 5 the branch may legitimately differ and the case is skipped."""
    from oracle import novak_oracle as O
    h = B.Handle(lr=lr, beta1=beta1, beta2=beta2, eps=1e-8, weight_decay=wd,
                 nesterov_variant=B.NOVAK_NESTEROV_APPROX, lookahead_k=k, lookahead_alpha=0.5)
    h.set_option(B.NOVAK_OPT_RECTIFIED, 1 if rectified else 0)
    h.set_option(B.NOVAK_OPT_ADAPTIVE_BETA, 1 if adaptive else 0)
    o = O.Oracle(O.Config(lr=lr, beta1=beta1, beta2=beta2, weight_decay=wd, lookahead_k=k,
                          rectified=rectified, adaptive_beta=adaptive), [np.zeros(1)])
    a, b = h.plan(t), o.scalars(t)
    h.destroy()
    if abs(b.rho_t - 5.0) < 1e-6:
        return
    assert a.rect_branch == b.rect_branch and a.is_sync == b.is_sync
    for name in ("bc1", "bc2", "rho_inf", "decay", "beta1_t", "beta2_t"):
        x, y = getattr(a, name), getattr(b, name)
        assert abs(x - y) <= 1e-11 * abs(y) + 1e-300, (name, x, y)
    # rho_t = rho_inf - 2 t beta2^t / (1 - beta2^t) cancels: compare at the scale of rho_inf
    assert abs(a.rho_t - b.rho_t) <= 1e-9 * max(1.0, b.rho_inf)
    if a.rect_branch:
        # r_t is well conditioned away from rho_t = 4 (the branch needs rho_t >= 5)
        assert abs(a.r_t - b.r_t) <= 1e-7 * b.r_t
        assert abs(a.step_size - b.step_size) <= 1e-7 * b.step_size
    else:
        assert a.r_t == 1.0 == b.r_t and abs(a.step_size - b.step_size) <= 1e-12 * b.step_size


@settings(max_examples=300, deadline=None)
@given(bits=st.lists(st.integers(0, 2 ** 32 - 1), min_size=1, max_size=64))
def test_oracle_bf16_rounding_equals_the_library_conversion_on_any_bit_pattern(bits):
    """Every finite fp32 bit pattern (subnormals, ties, values next to overflow): the
    oracle's nearest-even bfloat16 rounding against torch's fp32 -> bfloat16 conversion."""
    import torch
    from oracle import novak_oracle as O
    lib = O.default_library()
    x = np.array(bits, dtype=np.uint32).view(np.float32)
    x = x[np.isfinite(x)]
    if x.size == 0:
        return
    want = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([lib.novak_oracle_round_bf16(float(v)) for v in x])
    assert np.array_equal(got, want) and np.array_equal(np.signbit(got), np.signbit(want))
