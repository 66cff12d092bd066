"""Pins of the CPU oracle: each function checks the oracle loaded from ``lib`` against
something fixed by the paper or by mathematics, and raises AssertionError on a mismatch.

They take the library as an argument so that the same checks can be pointed at
deliberately broken builds of the oracle (see test_oracle_mutants.py).
"""
from __future__ import annotations

import os

import numpy as np

from oracle.ref import RefHPSGD, RefHPSGDAccum

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ worked examples
def parse_worked(path):
    mu, w0, grads, cases = None, None, {}, []
    for line in open(path):
        line = line.split("#", 1)[0].split()
        if not line:
            continue
        if line[0] == "mu":
            mu = float(line[1])
        elif line[0] == "w0":
            w0 = [float(x) for x in line[1:]]
        elif line[0] == "g":
            grads[(int(line[1]), int(line[2]))] = [float(x) for x in line[3:]]
        elif line[0] == "case":
            cases.append({"beta": float(line[2]), "lambda": float(line[4]),
                          "staleness": int(line[6]), "r": {}, "D": {}, "w": {}})
        elif line[0] == "r":
            cases[-1]["r"][(int(line[1]), int(line[2]))] = [float(x) for x in line[3:]]
        elif line[0] in ("D", "w"):
            cases[-1][line[0]][int(line[1])] = [float(x) for x in line[2:]]
    return mu, w0, grads, cases


def pin_worked_examples(lib):
    """Hand-worked K=2, P=4 rounds (Algorithm 2 + Algorithm 3 + Eq. 1), exact values."""
    mu, w0, grads, cases = parse_worked(os.path.join(GOLDEN, "worked_k2_p4.txt"))
    assert len(cases) == 6
    for c in cases:
        o = RefHPSGD(4, 2, mu, c["beta"], c["lambda"], c["staleness"], lib=lib)
        o.set_global(w0)
        for t in range(3):
            for i in range(2):
                o.local_step(i, np.array(grads[(t, i)], dtype=np.float32))
                np.testing.assert_array_equal(o.get_replica(i), np.float32(c["r"][(t, i)]),
                                              err_msg="replica, case %r round %d worker %d" % (c, t, i))
            o.sync_merge()
            np.testing.assert_array_equal(o.get_pending(), np.float32(c["D"][t]))
            np.testing.assert_array_equal(o.get_global(), np.float32(c["w"][t]))
        o.close()


# ------------------------------------------------------------------ Eq. 1 and Eq. 2 over uneven periods
def _periods(rng, syncs):
    """Local steps per synchronisation period: one before the first synchronisation, then a
    random number (the synchronising process stays busy for a while, Section 3.2)."""
    return [1] + [int(rng.integers(1, 5)) for _ in range(syncs - 1)]


def pin_eq1_eq2_over_uneven_periods(lib):
    """Plain SGD with several local steps per period, against the two closed forms the paper
    gives, evaluated in binary64 from the raw gradients:
      Eq. 1  the global model after synchronisation s is w_0 minus mu/n times ALL gradients of
             the periods that ended at synchronisations 0..s-1 (one synchronisation late);
      Eq. 2  inside a period, replica i is the global model minus mu times worker i's own
             gradients of that period, and the mean of the replicas minus w is the change the
             synchronisation puts aside."""
    rng = _rng(7)
    for trial in range(12):
        K = int(rng.integers(1, 6))
        P = int(rng.integers(1, 9))
        syncs = int(rng.integers(2, 7))
        steps = _periods(rng, syncs)
        mu = float(rng.choice([0.5, 0.1, 0.03]))
        mu64 = np.float64(np.float32(mu))
        w0 = rng.uniform(-1, 1, P).astype(np.float32)
        o = RefHPSGD(P, K, mu, 0.0, 0.0, 1, lib=lib)
        o.set_global(w0)
        landed = np.zeros(P)              # sum over workers and epochs of the periods already committed
        waiting = None                    # the same sum for the period reduced at the last synchronisation
        for s in range(syncs):
            own = np.zeros((K, P))        # each worker's gradients of the running period
            w_now = o.get_global().astype(np.float64)
            for h in range(steps[s]):
                for i in range(K):
                    g = rng.uniform(-1, 1, P).astype(np.float32)
                    o.local_step(i, g)
                    own[i] += g
                    np.testing.assert_allclose(o.get_replica(i), w_now - mu64 * own[i], rtol=0, atol=4e-6,
                                               err_msg="Eq. 2 replica, trial %d period %d step %d worker %d" % (trial, s, h, i))
            mean_change = np.mean([o.get_replica(i).astype(np.float64) for i in range(K)], axis=0) - w_now
            o.sync_merge()
            if waiting is not None:
                landed += waiting
            waiting = own.sum(axis=0)
            np.testing.assert_allclose(o.get_global(), w0.astype(np.float64) - mu64 / K * landed, rtol=0, atol=4e-6,
                                       err_msg="Eq. 1 global model after synchronisation %d (trial %d)" % (s, trial))
            np.testing.assert_allclose(o.get_pending(), mean_change, rtol=0, atol=4e-6)
            np.testing.assert_allclose(o.get_pending(), -mu64 / K * waiting, rtol=0, atol=4e-6)
        o.close()


# ------------------------------------------------------------------ closed form of Eq. 1
def pin_closed_form_eq1(lib):
    """Plain SGD, one-synchronisation delay: w_T = w_0 - mu/K * sum_i sum_{t<=T-2} g_i^t."""
    rng = _rng(11)
    K, P, T, mu = 4, 257, 10, 0.01
    w0 = rng.uniform(-0.1, 0.1, P).astype(np.float32)
    g = (rng.uniform(-1, 1, (T, K, P)) * 1e-2).astype(np.float32)
    o = RefHPSGD(P, K, mu, lib=lib)
    o.set_global(w0)
    for t in range(T):
        for i in range(K):
            o.local_step(i, g[t, i])
        o.sync_merge()
        upto = t - 1                                   # rounds 0..t-1 have been committed
        want = w0.astype(np.float64) - np.float64(np.float32(mu)) / K * g[:upto + 1].astype(np.float64).sum(axis=(0, 1))
        np.testing.assert_allclose(o.get_global(), want, rtol=1e-5, atol=1e-8)
    o.close()


# ------------------------------------------------------------------ K = 1 is an ordinary optimiser
def pin_k1_matches_library_sgd(lib):
    """K=1, staleness 0: the global model follows torch.optim.SGD (momentum, weight decay)."""
    import torch
    rng = _rng(13)
    P, T = 193, 25
    for lr, beta, lam in ((0.01, 0.0, 0.0), (0.1, 0.9, 0.0), (0.1, 0.9, 5e-4), (0.05, 0.5, 0.01)):
        w0 = rng.uniform(-0.1, 0.1, P).astype(np.float32)
        g = (rng.standard_normal((T, P)) * 1e-2).astype(np.float32)
        p = torch.nn.Parameter(torch.tensor(w0, dtype=torch.float64))
        opt = torch.optim.SGD([p], lr=float(np.float32(lr)), momentum=float(np.float32(beta)),
                              weight_decay=float(np.float32(lam)))
        o = RefHPSGD(P, 1, lr, beta, lam, 0, lib=lib)
        o.set_global(w0)
        for t in range(T):
            p.grad = torch.tensor(g[t], dtype=torch.float64)
            opt.step()
            o.local_step(0, g[t])
            o.sync_merge()
            np.testing.assert_allclose(o.get_global(), p.detach().numpy(), rtol=2e-5, atol=1e-7,
                                       err_msg="step %d lr %g beta %g lambda %g" % (t, lr, beta, lam))
        o.close()


# ------------------------------------------------------------------ Local SGD (Algorithm 1)
def pin_local_sgd_model_average(lib):
    """staleness 0, gamma local steps: the global model is the mean of the local models."""
    rng = _rng(17)
    K, P, gamma, loops, mu = 5, 64, 4, 3, 0.05
    w0 = rng.uniform(-1, 1, P).astype(np.float32)
    g = rng.uniform(-1, 1, (loops, gamma, K, P)).astype(np.float32)
    o = RefHPSGD(P, K, mu, 0.0, 0.0, 0, lib=lib)
    o.set_global(w0)
    w = w0.astype(np.float64)
    for l in range(loops):
        local = np.repeat(w[None, :], K, axis=0)
        for e in range(gamma):
            for i in range(K):
                o.local_step(i, g[l, e, i])
                local[i] -= np.float64(np.float32(mu)) * g[l, e, i]
        o.sync_merge()
        w = local.mean(axis=0)                          # AllReduce(model) / n
        np.testing.assert_allclose(o.get_global(), w, rtol=0, atol=3e-6)
    o.close()


# ------------------------------------------------------------------ Eq. 1 == Eq. 2 and invariants
def _ulp_distance(a, b):
    a = np.ascontiguousarray(a, dtype=np.float32).view(np.int32).astype(np.int64)
    b = np.ascontiguousarray(b, dtype=np.float32).view(np.int32).astype(np.int64)
    a = np.where(a < 0, -(a & 0x7FFFFFFF), a)
    b = np.where(b < 0, -(b & 0x7FFFFFFF), b)
    return np.abs(a - b)


def pin_eq1_equals_eq2(lib):
    """staleness 0: committing the averaged change equals averaging the replicas (Eq. 2)."""
    rng = _rng(19)
    K, P, mu = 7, 500, 0.1
    for beta in (0.0, 0.9):
        w0 = rng.uniform(-0.1, 0.1, P).astype(np.float32)
        o = RefHPSGD(P, K, mu, beta, 0.0, 0, lib=lib)
        o.set_global(w0)
        for t in range(4):
            for i in range(K):
                o.local_step(i, (rng.standard_normal(P) * 1e-2).astype(np.float32))
            mean_r = np.mean([o.get_replica(i).astype(np.float64) for i in range(K)], axis=0)
            o.sync_merge()
            np.testing.assert_allclose(o.get_global(), mean_r, rtol=0, atol=5e-8)
        o.close()


def pin_invariants(lib):
    rng = _rng(23)
    K, P, mu, beta = 6, 300, 0.1, 0.9
    w0 = rng.uniform(-0.1, 0.1, P).astype(np.float32)
    o = RefHPSGD(P, K, mu, beta, 5e-4, 1, lib=lib)
    o.set_global(w0)
    # replicas start as clones, momentum and pending change at zero
    for i in range(K):
        np.testing.assert_array_equal(o.get_replica(i), w0)
        np.testing.assert_array_equal(o.get_momentum(i), 0)
    np.testing.assert_array_equal(o.get_pending(), 0)
    for t in range(4):
        # worker K-1 sits this round out: its replica change is zero
        for i in range(K - 1):
            o.local_step(i, (rng.standard_normal(P) * 1e-2).astype(np.float32))
        w_before = o.get_global()
        d_before = o.get_pending()
        r_before = [o.get_replica(i) for i in range(K)]
        m_before = [o.get_momentum(i) for i in range(K)]
        np.testing.assert_array_equal(r_before[K - 1], w_before)
        o.sync_merge()
        assert o.merges == t + 1
        w_after = o.get_global()
        if t == 0:
            # the first synchronisation commits nothing (Algorithm 3 guard)
            np.testing.assert_array_equal(w_after, w0)
        else:
            np.testing.assert_array_equal(w_after, w_before + d_before)
        want_d = np.mean([r.astype(np.float64) - w_before for r in r_before], axis=0)
        np.testing.assert_allclose(o.get_pending(), want_d, rtol=1e-5, atol=1e-9)
        for i in range(K):
            np.testing.assert_array_equal(o.get_replica(i), w_after)        # clone of the latest global
            np.testing.assert_array_equal(o.get_momentum(i), m_before[i])   # merge leaves momentum alone
    o.close()


def pin_equal_gradients(lib):
    """Equal gradients on every worker: the merged change is one worker's change."""
    rng = _rng(29)
    P, mu = 400, 0.1
    for K in (2, 3, 8, 16):
        w0 = rng.uniform(-0.1, 0.1, P).astype(np.float32)
        o = RefHPSGD(P, K, mu, 0.9, 0.0, 1, lib=lib)
        one = RefHPSGD(P, 1, mu, 0.9, 0.0, 1, lib=lib)
        o.set_global(w0)
        one.set_global(w0)
        for t in range(3):
            g = (rng.standard_normal(P) * 1e-2).astype(np.float32)
            for i in range(K):
                o.local_step(i, g)
            one.local_step(0, g)
            change = o.get_replica(0) - o.get_global()      # one worker's change, exact in fp32 terms
            o.sync_merge()
            one.sync_merge()
            # a left-to-right sum of K equal terms is off by at most (K-1) roundings
            np.testing.assert_allclose(o.get_pending(), change, rtol=K * 6e-8, atol=1e-12)
            np.testing.assert_allclose(o.get_global(), one.get_global(), rtol=0, atol=1e-7)
        o.close()
        one.close()


def pin_staleness_is_one_sync_shift(lib):
    """Plain SGD: the delayed global after sync s+1 is the undelayed global after sync s."""
    rng = _rng(31)
    K, P, T, mu = 3, 100, 6, 0.05
    w0 = rng.uniform(-1, 1, P).astype(np.float32)
    g = rng.uniform(-1, 1, (T, K, P)).astype(np.float32)
    late = RefHPSGD(P, K, mu, 0.0, 0.0, 1, lib=lib)
    now = RefHPSGD(P, K, mu, 0.0, 0.0, 0, lib=lib)
    late.set_global(w0)
    now.set_global(w0)
    hist = []
    for t in range(T):
        for i in range(K):
            late.local_step(i, g[t, i])
            now.local_step(i, g[t, i])
        late.sync_merge()
        now.sync_merge()
        hist.append(now.get_global())
        want = w0 if t == 0 else hist[t - 1]
        np.testing.assert_allclose(late.get_global(), want, rtol=0, atol=2e-6)
    late.close()
    now.close()


def pin_storage_variants(lib):
    """bf16 storage == its exact widening; sparse rows == dense gradient with zero rows."""
    from workloads import hashgen
    rng = _rng(37)
    K, rows, cols, tail = 2, 9, 8, 21
    head = 13
    P = head + rows * cols + tail
    w0 = rng.uniform(-0.1, 0.1, P).astype(np.float32)
    for as_bf16 in (False, True):
        a = RefHPSGD(P, K, 0.1, 0.9, 1e-3, 1, lib=lib)
        b = RefHPSGD(P, K, 0.1, 0.9, 1e-3, 1, lib=lib)
        a.set_global(w0)
        b.set_global(w0)
        for t in range(3):
            for i in range(K):
                g = (rng.standard_normal(P) * 1e-2).astype(np.float32)
                active = np.sort(rng.choice(rows, size=3, replace=False)).astype(np.int32)
                seg = g[head:head + rows * cols].reshape(rows, cols).copy()
                dense_equiv = g.copy()
                mask = np.zeros(rows, dtype=bool)
                mask[active] = True
                dense_equiv[head:head + rows * cols].reshape(rows, cols)[~mask] = 0.0
                vals = seg[active]
                garbage = g.copy()
                garbage[head:head + rows * cols] = 123.0          # must be ignored
                if as_bf16:
                    a.local_step(i, hashgen.bf16_to_f32(hashgen.f32_to_bf16(dense_equiv)))
                    b.local_step_sparse(i, hashgen.f32_to_bf16(garbage), head, rows, cols, active,
                                        hashgen.f32_to_bf16(vals))
                else:
                    a.local_step(i, dense_equiv)
                    b.local_step_sparse(i, garbage, head, rows, cols, active, vals)
                np.testing.assert_array_equal(a.get_replica(i), b.get_replica(i))
                np.testing.assert_array_equal(a.get_momentum(i), b.get_momentum(i))
            a.sync_merge()
            b.sync_merge()
            np.testing.assert_array_equal(a.get_global(), b.get_global())
        if as_bf16:
            c = RefHPSGD(P, K, 0.1, 0.9, 1e-3, 1, lib=lib)
            c.set_global(w0)
            g = (rng.standard_normal(P) * 1e-2).astype(np.float32)
            bits = hashgen.f32_to_bf16(g)
            c.local_step(0, bits)
            a2 = RefHPSGD(P, K, 0.1, 0.9, 1e-3, 1, lib=lib)
            a2.set_global(w0)
            a2.local_step(0, hashgen.bf16_to_f32(bits))
            np.testing.assert_array_equal(c.get_replica(0), a2.get_replica(0))
            c.close()
            a2.close()
        a.close()
        b.close()


# ------------------------------------------------------------------ gradient-accumulation form
def pin_accum_worked_example(lib):
    """The printed form on the hand-worked plain-SGD rounds: same replicas and global model;
    the AllReduce result is the mean gradient, i.e. -D/mu of the replica-change form."""
    mu, w0, grads, cases = parse_worked(os.path.join(GOLDEN, "worked_k2_p4.txt"))
    c = [c for c in cases if c["beta"] == 0 and c["lambda"] == 0 and c["staleness"] == 1][0]
    o = RefHPSGDAccum(4, 2, mu, lib=lib)
    o.set_global(w0)
    for t in range(3):
        for i in range(2):
            o.local_step(i, np.array(grads[(t, i)], dtype=np.float32))
            np.testing.assert_array_equal(o.get_replica(i), np.float32(c["r"][(t, i)]))
        acc = [o.get_accumulated(i) for i in range(2)]
        np.testing.assert_array_equal(acc[0], np.float32(grads[(t, 0)]))
        o.sync_merge()
        np.testing.assert_array_equal(o.get_global(), np.float32(c["w"][t]))
        np.testing.assert_array_equal(o.get_synced(), -np.float32(c["D"][t]) / np.float32(mu))
        for i in range(2):
            np.testing.assert_array_equal(o.get_replica(i), o.get_global())
            np.testing.assert_array_equal(o.get_accumulated(i), 0)
    o.close()


def pin_accum_closed_form_and_replica_form(lib):
    """The printed form against the closed form of Eq. 1 in binary64 over uneven periods, and
    against the replica-change oracle (Eq. 1 == Eq. 2)."""
    rng = _rng(41)
    for trial in range(8):
        K = int(rng.integers(1, 6))
        P = int(rng.integers(1, 9))
        syncs = int(rng.integers(2, 7))
        steps = _periods(rng, syncs)
        mu = float(rng.choice([0.5, 0.1, 0.03]))
        w0 = rng.uniform(-1, 1, P).astype(np.float32)
        acc = RefHPSGDAccum(P, K, mu, lib=lib)
        rep = RefHPSGD(P, K, mu, 0.0, 0.0, 1, lib=lib)
        acc.set_global(w0)
        rep.set_global(w0)
        committed = np.zeros(P)
        period_sum = None
        for s in range(syncs):
            this_period = np.zeros(P)
            own = np.zeros((K, P))
            for _ in range(steps[s]):
                for i in range(K):
                    g = rng.uniform(-1, 1, P).astype(np.float32)
                    acc.local_step(i, g)
                    rep.local_step(i, g)
                    own[i] += g
                    this_period += g
            for i in range(K):
                np.testing.assert_allclose(acc.get_accumulated(i), own[i], rtol=0, atol=4e-6)
            if period_sum is not None:
                committed += period_sum                 # the previous period lands now
            period_sum = this_period
            acc.sync_merge()
            rep.sync_merge()
            closed = w0.astype(np.float64) - np.float64(np.float32(mu)) / K * committed
            np.testing.assert_allclose(acc.get_global(), closed, rtol=0, atol=4e-6)
            np.testing.assert_allclose(acc.get_global(), rep.get_global(), rtol=0, atol=4e-6)
            np.testing.assert_allclose(acc.get_synced(), this_period / K, rtol=1e-5, atol=1e-7)
            for i in range(K):
                np.testing.assert_array_equal(acc.get_replica(i), acc.get_global())
        acc.close()
        rep.close()


ALL_PINS = [
    pin_worked_examples,
    pin_eq1_eq2_over_uneven_periods,
    pin_closed_form_eq1,
    pin_k1_matches_library_sgd,
    pin_local_sgd_model_average,
    pin_eq1_equals_eq2,
    pin_invariants,
    pin_equal_gradients,
    pin_staleness_is_one_sync_shift,
    pin_storage_variants,
    pin_accum_worked_example,
    pin_accum_closed_form_and_replica_form,
]
