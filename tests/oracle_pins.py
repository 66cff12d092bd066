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


# ------------------------------------------------------------------ literal Algorithms 2 and 3
def literal_hpsgd(w0, grads, mu, busy):
    """Algorithms 2 and 3 as printed, in binary64, with explicit shared variables.

    ``grads[e][i]`` is worker i's local gradient at epoch e.  A synchronisation, once
    started, keeps P_s busy for ``busy`` further epochs.  All workers hold the same global
    model (one ``w``).  Returns the global model after every synchronisation start and the
    list of (epoch, worker, replica) seen in the synchronising branch.
    """
    n = len(grads[0])
    w = np.array(w0, dtype=np.float64)
    status = "idling"
    counter = 0
    busy_left = 0
    acc = [np.zeros_like(w) for _ in range(n)]          # accumulated gradients per worker
    replica = [None] * n
    synced = None                                       # result of the last AllReduce
    globals_after_sync, replicas_seen = [], []
    for e in range(len(grads)):
        if status == "synchronizing":
            for i in range(n):
                if counter == 0:
                    replica[i] = w.copy()                       # make replica
                replica[i] = replica[i] - mu * grads[e][i]      # update replica
                acc[i] = acc[i] + grads[e][i]                   # accumulate gradients
                replicas_seen.append((e, i, replica[i].copy()))
            counter += 1
            busy_left -= 1
            if busy_left == 0:
                counter = 0                                     # P_s: reset the counter
                status = "idling"                               # P_s: mark the status
        else:
            for i in range(n):
                acc[i] = acc[i] + grads[e][i]
            status = "synchronizing"
            # ---- StartSync(P_s): Algorithm 3
            if e - counter > 0:
                w = w - mu * synced                             # commit the previous AllReduce
            synced = sum(acc) / n                               # AllReduce, mean over workers
            acc = [np.zeros_like(w) for _ in range(n)]
            globals_after_sync.append(w.copy())
            if busy == 0:
                counter = 0
                status = "idling"
            else:
                busy_left = busy
    return globals_after_sync, replicas_seen


def pin_literal_algorithms(lib):
    """The replica-change oracle against the printed gradient-accumulation form (plain SGD)."""
    rng = _rng(7)
    for trial in range(12):
        K = int(rng.integers(1, 6))
        P = int(rng.integers(1, 9))
        busy = int(rng.integers(0, 4))
        syncs = int(rng.integers(2, 6))
        epochs = 1 + (syncs - 1) * (busy + 1)
        mu = float(rng.choice([0.5, 0.1, 0.03]))
        w0 = rng.uniform(-1, 1, P).astype(np.float32)
        grads = rng.uniform(-1, 1, (epochs, K, P)).astype(np.float32)
        want_w, want_r = literal_hpsgd(w0, grads.astype(np.float64), mu, busy)
        assert len(want_w) == syncs

        o = RefHPSGD(P, K, mu, 0.0, 0.0, 1, lib=lib)
        o.set_global(w0)
        e = 0
        seen = []
        for s in range(syncs):
            steps = 1 if s == 0 else busy + 1
            for h in range(steps):
                for i in range(K):
                    o.local_step(i, grads[e, i])
                    # the printed algorithm touches the replica only while P_s is busy,
                    # i.e. on every step of a period but its last one
                    if s > 0 and h < steps - 1:
                        seen.append((e, i, o.get_replica(i)))
                e += 1
            o.sync_merge()
            np.testing.assert_allclose(o.get_global(), want_w[s], rtol=0, atol=4e-6,
                                       err_msg="global after synchronisation %d (trial %d)" % (s, trial))
        assert len(seen) == len(want_r)
        for (e1, i1, r1), (e2, i2, r2) in zip(seen, want_r):
            assert (e1, i1) == (e2, i2)
            np.testing.assert_allclose(r1, r2, rtol=0, atol=4e-6)
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


def pin_accum_literal_and_closed_form(lib):
    """The printed form against its binary64 transcription with status/counter flags, the
    closed form of Eq. 1, and the replica-change oracle (Eq. 1 == Eq. 2)."""
    rng = _rng(41)
    for trial in range(8):
        K = int(rng.integers(1, 6))
        P = int(rng.integers(1, 9))
        busy = int(rng.integers(0, 4))
        syncs = int(rng.integers(2, 6))
        epochs = 1 + (syncs - 1) * (busy + 1)
        mu = float(rng.choice([0.5, 0.1, 0.03]))
        w0 = rng.uniform(-1, 1, P).astype(np.float32)
        grads = rng.uniform(-1, 1, (epochs, K, P)).astype(np.float32)
        want_w, _ = literal_hpsgd(w0, grads.astype(np.float64), mu, busy)
        acc = RefHPSGDAccum(P, K, mu, lib=lib)
        rep = RefHPSGD(P, K, mu, 0.0, 0.0, 1, lib=lib)
        acc.set_global(w0)
        rep.set_global(w0)
        e = 0
        committed = np.zeros(P)
        period_sum = None
        for s in range(syncs):
            steps = 1 if s == 0 else busy + 1
            this_period = np.zeros(P)
            for _ in range(steps):
                for i in range(K):
                    acc.local_step(i, grads[e, i])
                    rep.local_step(i, grads[e, i])
                this_period += grads[e].astype(np.float64).sum(axis=0)
                e += 1
            if period_sum is not None:
                committed += period_sum                 # the previous period lands now
            period_sum = this_period
            acc.sync_merge()
            rep.sync_merge()
            np.testing.assert_allclose(acc.get_global(), want_w[s], rtol=0, atol=4e-6)
            closed = w0.astype(np.float64) - np.float64(np.float32(mu)) / K * committed
            np.testing.assert_allclose(acc.get_global(), closed, rtol=0, atol=4e-6)
            np.testing.assert_allclose(acc.get_global(), rep.get_global(), rtol=0, atol=4e-6)
            np.testing.assert_allclose(acc.get_synced(), this_period / K, rtol=1e-5, atol=1e-7)
        acc.close()
        rep.close()


ALL_PINS = [
    pin_worked_examples,
    pin_literal_algorithms,
    pin_closed_form_eq1,
    pin_k1_matches_library_sgd,
    pin_local_sgd_model_average,
    pin_eq1_equals_eq2,
    pin_invariants,
    pin_equal_gradients,
    pin_staleness_is_one_sync_shift,
    pin_storage_variants,
    pin_accum_worked_example,
    pin_accum_literal_and_closed_form,
]
