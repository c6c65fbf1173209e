"""Checks that pin the CPU oracle to facts fixed outside of it.

Each ``pin_*`` function takes an optional handle to an oracle shared library
(``None`` = the committed one) and raises AssertionError when the oracle
disagrees with a closed form, a library routine, a brute-force enumeration or
a structural invariant.  The same functions are run against deliberately
broken copies of the oracle (tests/test_oracle_mutants.py) to show that a
plausible mistake anywhere in it trips at least one of them.

None of the expected values below is produced by the oracle's own recurrence:
they come from algebra (geometric series, cumulative sums), from numpy / scipy
routines, or from explicit O(T^2) products.
"""

from __future__ import annotations

import math

import numpy as np
import scipy.signal

import oracle

BIG_Z = 40.0  # z/(1+exp(-z)) == z to 4e-18 relative: the gate becomes a known factor


def _close(a, b, rtol=1e-11, atol=1e-13, what=""):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    if a.shape != b.shape or not np.allclose(a, b, rtol=rtol, atol=atol):
        err = np.max(np.abs(a - b)) if a.shape == b.shape else float("inf")
        raise AssertionError(f"{what}: max abs diff {err}")


def _identity_conv(Dn, W):
    w = np.zeros((Dn, W))
    w[:, W - 1] = 1.0
    return w


def _rng(i):
    return np.random.default_rng(1000 + i)


# ------------------------------------------------------------------ scalar functions
def pin_scalar_functions(L=None):
    l = L or oracle.lib()
    silu, sp = l.mdo_silu, l.mdo_softplus
    assert silu(0.0) == 0.0
    # sigmoid(1) to 16 digits (textbook constant) => SiLU(1)
    _close(silu(1.0), 0.7310585786300049, what="SiLU(1)")
    _close(silu(-1.0), -0.2689414213699951, what="SiLU(-1)")
    for v in (0.3, 2.0, 7.5):
        _close(silu(v) - silu(-v), v, what="SiLU(v)-SiLU(-v)=v")
    _close(silu(50.0), 50.0, rtol=1e-15, what="SiLU(v)->v")
    _close(sp(0.0), math.log(2.0), what="softplus(0)")
    for v in (0.1, 1.0, 5.0):
        _close(sp(v) - sp(-v), v, what="softplus(v)-softplus(-v)=v")
    _close(sp(40.0), 40.0, rtol=1e-15, what="softplus(v)->v")
    _close(sp(-30.0), math.exp(-30.0), rtol=1e-12, atol=0, what="softplus(v)->exp(v)")
    # derivative of softplus is the logistic function
    eps = 1e-6
    _close((sp(0.7 + eps) - sp(0.7 - eps)) / (2 * eps), 1.0 / (1.0 + math.exp(-0.7)), rtol=1e-8, what="softplus'")


# ------------------------------------------------------------------ recurrence, closed forms
def pin_geometric_series(L=None):
    """Constant Delta, A, B, C, u and a given h0:
    h_t = a^t h0 + b (1-a^t)/(1-a), a = exp(Delta A), b = Delta B u."""
    g = _rng(1)
    Dn, N, T, W = 3, 4, 37, 4
    A = -g.uniform(0.2, 3.0, (Dn, N))
    Dsk = g.normal(size=Dn)
    delta = g.uniform(0.01, 0.3, Dn)
    u = g.normal(size=Dn)
    Bc = g.normal(size=N)
    Cc = g.normal(size=N)
    h0 = g.normal(size=(1, Dn, N))
    lay = oracle.Layer(A, Dsk, _identity_conv(Dn, W), None, None, flags=oracle.PRECONV)
    x = np.tile(u, (T, 1)); dt = np.tile(delta, (T, 1)); z = np.full((T, Dn), BIG_Z)
    out, _, hT = oracle.prefill(lay, x, z, dt, np.tile(Bc, (T, 1)), np.tile(Cc, (T, 1)), h_init=h0, _lib_override=L)
    a = np.exp(delta[:, None] * A)                     # (D,N)
    b = delta[:, None] * Bc[None, :] * u[:, None]      # (D,N)
    t = np.arange(1, T + 1)[:, None, None]
    h = a[None] ** t * h0 + b[None] * (1 - a[None] ** t) / (1 - a[None])
    y = (h * Cc[None, None, :]).sum(-1) + Dsk[None, :] * u[None, :]
    _close(out, y * BIG_Z, what="geometric series: out")
    _close(hT[0], h[-1], what="geometric series: final state")


def pin_cumulative_sum(L=None):
    """A = 0 exactly: h_t = sum_{s<=t} Delta_s B_s u_s."""
    g = _rng(2)
    Dn, N, T, W = 2, 3, 29, 4
    lay = oracle.Layer(np.zeros((Dn, N)), np.zeros(Dn), _identity_conv(Dn, W), None, None, flags=oracle.PRECONV)
    u = g.normal(size=(T, Dn)); delta = g.uniform(0.0, 0.5, (T, Dn))
    B = g.normal(size=(T, N)); Cm = g.normal(size=(T, N))
    out, _, hT = oracle.prefill(lay, u, np.full((T, Dn), BIG_Z), delta, B, Cm, _lib_override=L)
    h = np.cumsum((delta * u)[:, :, None] * B[:, None, :], axis=0)     # (T,D,N)
    _close(hT[0], h[-1], what="A=0: final state is the cumulative sum")
    _close(out, (h * Cm[:, None, :]).sum(-1) * BIG_Z, what="A=0: out")


def pin_frozen_state(L=None):
    """Delta = 0: the state never moves and y_t = C_t.h0 + D u_t."""
    g = _rng(3)
    Dn, N, T, W = 3, 5, 11, 4
    A = -g.uniform(0.5, 2.0, (Dn, N)); Dsk = g.normal(size=Dn)
    lay = oracle.Layer(A, Dsk, _identity_conv(Dn, W), None, None, flags=oracle.PRECONV)
    u = g.normal(size=(T, Dn)); Cm = g.normal(size=(T, N)); B = g.normal(size=(T, N))
    h0 = g.normal(size=(1, Dn, N))
    out, _, hT = oracle.prefill(lay, u, np.full((T, Dn), BIG_Z), np.zeros((T, Dn)), B, Cm, h_init=h0, _lib_override=L)
    _close(hT, h0, rtol=0, atol=0, what="Delta=0: state frozen")
    _close(out, (np.einsum("tn,dn->td", Cm, h0[0]) + Dsk[None] * u) * BIG_Z, what="Delta=0: out")


def pin_brute_force(L=None):
    """Tiny case by explicit O(T^2) products:
    h_T = (prod_r a_r) h0 + sum_s (prod_{r>s} a_r) b_s, no running state."""
    g = _rng(4)
    Dn, N, T, W = 2, 2, 7, 4
    A = -g.uniform(0.3, 2.0, (Dn, N)); Dsk = g.normal(size=Dn)
    lay = oracle.Layer(A, Dsk, _identity_conv(Dn, W), None, None, flags=oracle.PRECONV)
    u = g.normal(size=(T, Dn)); delta = g.uniform(0.01, 0.6, (T, Dn))
    B = g.normal(size=(T, N)); Cm = g.normal(size=(T, N)); z = g.normal(size=(T, Dn))
    h0 = g.normal(size=(1, Dn, N))
    out, _, hT = oracle.prefill(lay, u, z, delta, B, Cm, h_init=h0, _lib_override=L)
    exp_out = np.zeros((T, Dn))
    for d in range(Dn):
        for t in range(T):
            y = Dsk[d] * u[t, d]
            for n in range(N):
                h = h0[0, d, n] * math.prod(math.exp(delta[r, d] * A[d, n]) for r in range(t + 1))
                for s in range(t + 1):
                    w = math.prod(math.exp(delta[r, d] * A[d, n]) for r in range(s + 1, t + 1))
                    h += w * delta[s, d] * B[s, n] * u[s, d]
                y += Cm[t, n] * h
                if t == T - 1:
                    _close(hT[0, d, n], h, what="brute force: state")
            sig = 1.0 / (1.0 + math.exp(-z[t, d]))
            exp_out[t, d] = y * z[t, d] * sig
    _close(out, exp_out, what="brute force: out")


def pin_iir_filter(L=None):
    """Constant Delta, B, C and a varying input: each (d,n) is the one-pole
    filter h_t = a h_{t-1} + b u_t, i.e. scipy.signal.lfilter([b],[1,-a],u)."""
    g = _rng(5)
    Dn, N, T, W = 2, 3, 64, 4
    A = -g.uniform(0.2, 2.0, (Dn, N))
    delta = g.uniform(0.05, 0.4, Dn); Bc = g.normal(size=N); Cc = g.normal(size=N)
    lay = oracle.Layer(A, np.zeros(Dn), _identity_conv(Dn, W), None, None, flags=oracle.PRECONV)
    u = g.normal(size=(T, Dn))
    out, _, hT = oracle.prefill(lay, u, np.full((T, Dn), BIG_Z), np.tile(delta, (T, 1)),
                                np.tile(Bc, (T, 1)), np.tile(Cc, (T, 1)), _lib_override=L)
    y = np.zeros((T, Dn))
    for d in range(Dn):
        for n in range(N):
            a = math.exp(delta[d] * A[d, n]); b = delta[d] * Bc[n]
            hf = scipy.signal.lfilter([b], [1.0, -a], u[:, d])
            y[:, d] += Cc[n] * hf
            _close(hT[0, d, n], hf[-1], what="lfilter: state")
    _close(out, y * BIG_Z, what="lfilter: out")


def pin_softplus_and_bias_in_path(L=None):
    """Delta = softplus(dt + dt_bias): choose dt + bias = log(expm1(0.05)) so that
    Delta = 0.05 is known, then use the geometric closed form for one step count."""
    Dn, N, T, W = 2, 2, 9, 4
    A = -np.array([[1.0, 2.0], [0.5, 3.0]]); target = 0.05
    pre = math.log(math.expm1(target))
    bias = np.array([0.7, -1.3]); dt = np.tile(pre - bias, (T, 1))
    lay = oracle.Layer(A, np.zeros(Dn), _identity_conv(Dn, W), None, bias, flags=oracle.PRECONV | oracle.DT_SOFTPLUS)
    out, _, hT = oracle.prefill(lay, np.ones((T, Dn)), np.full((T, Dn), BIG_Z), dt, np.ones((T, N)), np.ones((T, N)), _lib_override=L)
    a = np.exp(target * A)
    h = target * (1 - a ** T) / (1 - a)
    _close(hT[0], h, rtol=1e-10, what="softplus+bias: state")
    # pass-through mode: Delta = dt + bias, no activation
    lay2 = oracle.Layer(A, np.zeros(Dn), _identity_conv(Dn, W), None, bias, flags=oracle.PRECONV)
    _, _, hT2 = oracle.prefill(lay2, np.ones((T, Dn)), np.full((T, Dn), BIG_Z), np.tile(target - bias, (T, 1)),
                               np.ones((T, N)), np.ones((T, N)), _lib_override=L)
    _close(hT2[0], h, rtol=1e-10, what="pass-through Delta: state")


# ------------------------------------------------------------------ convolution
def pin_conv_impulse(L=None):
    """A unit impulse at t0 meets tap W-1 first, then W-2, ... (cross-correlation,
    tap W-1 on the current token).  Taps are large so that SiLU(v) = v to 1e-10."""
    Dn, N, W, T, t0 = 2, 1, 4, 12, 5
    w = np.array([[25.0, 30.0, 35.0, 40.0], [41.0, 33.0, 29.0, 26.0]])
    lay = oracle.Layer(np.zeros((Dn, N)), None, w, None, None, flags=oracle.CONV_ONLY)
    x = np.zeros((T, Dn)); x[t0] = 1.0
    zeros = np.zeros((T, Dn)); zn = np.zeros((T, N))
    out, conv_f, _ = oracle.prefill(lay, x, zeros, zeros, zn, zn, _lib_override=L)
    exp_u = np.zeros((T, Dn))
    for j in range(W):
        exp_u[t0 + j] = w[:, W - 1 - j]
    _close(out, exp_u, rtol=1e-9, what="conv impulse response")
    # window after the last token holds the last W-1 raw inputs, oldest first
    x2 = np.arange(1.0, T * Dn + 1).reshape(T, Dn)
    _, conv_f, _ = oracle.prefill(lay, x2, zeros, zeros, zn, zn, _lib_override=L)
    _close(conv_f[0], x2[-(W - 1):], rtol=0, atol=0, what="conv window contents")


def pin_conv_numpy(L=None):
    """General input against numpy.convolve; a bias of 50 keeps SiLU(v) = v to 1e-20."""
    g = _rng(6)
    Dn, N, W, T = 3, 1, 4, 40
    w = g.normal(scale=0.5, size=(Dn, W)); b = np.full(Dn, 50.0) + g.normal(size=Dn)
    lay = oracle.Layer(np.zeros((Dn, N)), None, w, b, None, flags=oracle.CONV_ONLY)
    x = g.normal(size=(T, Dn)); zeros = np.zeros((T, Dn)); zn = np.zeros((T, N))
    out, _, _ = oracle.prefill(lay, x, zeros, zeros, zn, zn, _lib_override=L)
    for d in range(Dn):
        ref = np.convolve(x[:, d], w[d, ::-1])[:T] + b[d]
        _close(out[:, d], ref, rtol=1e-12, what="conv vs numpy.convolve")
    # with a cached window: same as convolving the window followed by x
    ci = g.normal(size=(1, W - 1, Dn))
    out2, _, _ = oracle.prefill(lay, x, zeros, zeros, zn, zn, conv_init=ci, _lib_override=L)
    for d in range(Dn):
        xx = np.concatenate([ci[0, :, d], x[:, d]])
        ref = np.convolve(xx, w[d, ::-1])[W - 1:W - 1 + T] + b[d]
        _close(out2[:, d], ref, rtol=1e-12, what="conv with cached window")


def pin_conv_feeds_recurrence(L=None):
    """Full path == split path: u from the conv-only mode, fed to the
    pre-convolved mode, gives the same out and state; and u (not x) is what the
    skip term D*u uses (A = 0, B = 0 isolates it)."""
    g = _rng(7)
    Dn, N, W, T = 3, 2, 4, 17
    A = -g.uniform(0.3, 2.0, (Dn, N)); Dsk = g.normal(size=Dn); w = g.normal(scale=0.5, size=(Dn, W)); cb = g.normal(size=Dn)
    bias = g.normal(size=Dn) - 3
    x = g.normal(size=(T, Dn)); z = g.normal(size=(T, Dn)); dt = g.normal(size=(T, Dn))
    B = g.normal(size=(T, N)); Cm = g.normal(size=(T, N))
    full = oracle.Layer(A, Dsk, w, cb, bias, flags=oracle.DT_SOFTPLUS)
    out, cf, hf = oracle.prefill(full, x, z, dt, B, Cm, _lib_override=L)
    u, cf2, _ = oracle.prefill(full, x, z, dt, B, Cm, flags=oracle.DT_SOFTPLUS | oracle.CONV_ONLY, _lib_override=L)
    out2, _, hf2 = oracle.prefill(full, u, z, dt, B, Cm, flags=oracle.DT_SOFTPLUS | oracle.PRECONV, _lib_override=L)
    _close(out2, out, rtol=0, atol=0, what="split mode == fused mode (out)")
    _close(hf2, hf, rtol=0, atol=0, what="split mode == fused mode (state)")
    _close(cf2, cf, rtol=0, atol=0, what="conv window identical in both modes")
    skip = oracle.Layer(np.zeros((Dn, N)), Dsk, w, cb, bias, flags=oracle.DT_SOFTPLUS)
    out3, _, _ = oracle.prefill(skip, x, np.full((T, Dn), BIG_Z), dt, np.zeros((T, N)), Cm, _lib_override=L)
    _close(out3, Dsk[None] * u * BIG_Z, what="skip term uses the conv output")


# ------------------------------------------------------------------ structure
def _random_problem(i, Dn=4, N=3, W=4, T=23, conv_bias=True):
    g = _rng(i)
    A = -g.uniform(0.3, 4.0, (Dn, N)); Dsk = g.normal(size=Dn); w = g.normal(scale=0.5, size=(Dn, W))
    cb = g.normal(size=Dn) if conv_bias else None
    bias = g.normal(size=Dn) - 3
    lay = oracle.Layer(A, Dsk, w, cb, bias, flags=oracle.DT_SOFTPLUS)
    x = g.normal(size=(T, Dn)); z = g.normal(size=(T, Dn)); dt = g.normal(size=(T, Dn))
    B = g.normal(size=(T, N)); Cm = g.normal(size=(T, N))
    return lay, x, z, dt, B, Cm


def pin_prefill_handoff(L=None):
    """prefill(L) == prefill(L1) -> carried state -> prefill(L - L1), including L1 < W-1."""
    lay, x, z, dt, B, Cm = _random_problem(8)
    T = x.shape[0]
    out, cf, hf = oracle.prefill(lay, x, z, dt, B, Cm, _lib_override=L)
    for L1 in (1, 2, 3, 4, 11, T - 1):
        o1, c1, h1 = oracle.prefill(lay, x[:L1], z[:L1], dt[:L1], B[:L1], Cm[:L1], _lib_override=L)
        o2, c2, h2 = oracle.prefill(lay, x[L1:], z[L1:], dt[L1:], B[L1:], Cm[L1:], conv_init=c1, h_init=h1, _lib_override=L)
        _close(np.concatenate([o1, o2]), out, rtol=0, atol=0, what=f"hand-off at {L1}: out")
        _close(c2, cf, rtol=0, atol=0, what=f"hand-off at {L1}: conv window")
        _close(h2, hf, rtol=0, atol=0, what=f"hand-off at {L1}: state")


def pin_prefill_equals_chain(L=None):
    """prefill(L+k) == prefill(L) followed by a k-node chain through the tree routine."""
    lay, x, z, dt, B, Cm = _random_problem(9)
    T, k = x.shape[0], 5
    out, cf, hf = oracle.prefill(lay, x, z, dt, B, Cm, _lib_override=L)
    L0 = T - k
    _, c0, h0 = oracle.prefill(lay, x[:L0], z[:L0], dt[:L0], B[:L0], Cm[:L0], _lib_override=L)
    parents = np.arange(-1, k - 1)
    to, tc, th = oracle.tree(lay, parents, x[L0:], z[L0:], dt[L0:], B[L0:], Cm[L0:], conv0=c0[0], h0=h0[0], _lib_override=L)
    _close(to, out[L0:], rtol=0, atol=0, what="chain == prefill tail (out)")
    _close(tc[-1], cf[0], rtol=0, atol=0, what="chain == prefill tail (conv window)")
    _close(th[-1], hf[0], rtol=0, atol=0, what="chain == prefill tail (state)")


def pin_tree_paths(L=None):
    """Every node equals its root-to-node path run as one short sequence through
    the prefill routine; siblings fed identical inputs agree bit for bit."""
    lay, x, z, dt, B, Cm = _random_problem(10, T=15)
    g = _rng(11)
    parents = np.array([-1, 0, 0, 1, 1, 2, 2, 3, 3, 4, 4, 5, 5, 6, 6])
    Dn, N, W = lay.dims
    c0 = g.normal(size=(W - 1, Dn)); h0 = g.normal(size=(Dn, N))
    # make nodes 3 and 4 (children of 1) identical twins
    for a in (x, z, dt, B, Cm):
        a[4] = a[3]
    to, tc, th = oracle.tree(lay, parents, x, z, dt, B, Cm, conv0=c0, h0=h0, _lib_override=L)
    for v in range(len(parents)):
        path = []
        a = v
        while a >= 0:
            path.append(a); a = parents[a]
        path = path[::-1]
        po, pc, ph = oracle.prefill(lay, x[path], z[path], dt[path], B[path], Cm[path],
                                    conv_init=c0[None], h_init=h0[None], _lib_override=L)
        _close(to[v], po[-1], rtol=0, atol=0, what=f"node {v}: out")
        _close(tc[v], pc[0], rtol=0, atol=0, what=f"node {v}: conv window")
        _close(th[v], ph[0], rtol=0, atol=0, what=f"node {v}: state")
    _close(to[3], to[4], rtol=0, atol=0, what="twin siblings")
    _close(th[3], th[4], rtol=0, atol=0, what="twin siblings (state)")
    # a child really continues from its parent: its window's last row is its own input
    _close(tc[:, -1, :], x, rtol=0, atol=0, what="node window ends with the node's input")
    _close(tc[1:, -2, :], x[parents[1:]], rtol=0, atol=0, what="node window holds the parent's input")


def pin_varlen(L=None):
    """Packed sequences == each sequence alone (state and window reset per sequence)."""
    lay, x, z, dt, B, Cm = _random_problem(12, T=31)
    cu = np.array([0, 2, 9, 10, 31], dtype=np.int32)
    g = _rng(13)
    Dn, N, W = lay.dims
    S = len(cu) - 1
    ci = g.normal(size=(S, W - 1, Dn)); hi = g.normal(size=(S, Dn, N))
    out, cf, hf = oracle.prefill(lay, x, z, dt, B, Cm, cu_seqlens=cu, conv_init=ci, h_init=hi, _lib_override=L)
    for s in range(S):
        a, b = cu[s], cu[s + 1]
        o, c, h = oracle.prefill(lay, x[a:b], z[a:b], dt[a:b], B[a:b], Cm[a:b], conv_init=ci[s:s + 1], h_init=hi[s:s + 1], _lib_override=L)
        _close(out[a:b], o, rtol=0, atol=0, what=f"varlen seq {s}: out")
        _close(cf[s], c[0], rtol=0, atol=0, what=f"varlen seq {s}: window")
        _close(hf[s], h[0], rtol=0, atol=0, what=f"varlen seq {s}: state")
    # a 1-token and a 2-token sequence shift the cached window instead of replacing it
    _close(cf[2, :2], ci[2, 1:], rtol=0, atol=0, what="1-token sequence shifts the window by one")
    _close(cf[0, :1], ci[0, 2:], rtol=0, atol=0, what="2-token sequence shifts the window by two")


def _proj_problem(i, Dn=6, N=3, R=2, M=9):
    """Random tree problem for the projection pins; dense weights, every node with its own inputs."""
    lay, x, z, _, _, _ = _random_problem(i, Dn=Dn, N=N, T=M)
    g = _rng(100 + i)
    Wx = g.normal(size=(R + 2 * N, Dn)); Wdt = g.normal(size=(Dn, R))
    parents = np.array([-1, 0, 0, 1, 1, 2, 3, 3, 6][:M])
    W = lay.dims[2]
    c0 = g.normal(size=(W - 1, Dn)); h0 = g.normal(size=(Dn, N))
    return lay, Wx, Wdt, parents, x, z, c0, h0


def pin_proj_library_matmul(L=None):
    """The projection tree == the plain tree fed with step size, B and C computed by numpy's matmul from the conv
    outputs (conv outputs from the conv-only tree, itself pinned by the conv pins)."""
    lay, Wx, Wdt, parents, x, z, c0, h0 = _proj_problem(20)
    Dn, N, W = lay.dims
    R = Wdt.shape[1]
    out, cn, hn, dt, B, Cm = oracle.tree_proj(lay, Wx, Wdt, parents, x, z, conv0=c0, h0=h0, _lib_override=L)
    zero = np.zeros_like(x); zbc = np.zeros((len(parents), N))
    u, cu_nodes, _ = oracle.tree(lay, parents, x, zero, zero, zbc, zbc, conv0=c0, h0=h0, flags=lay.flags | oracle.CONV_ONLY, _lib_override=L)
    s = np.matmul(u, Wx.T)
    dt_ref = np.matmul(s[:, :R], Wdt.T)
    _close(dt, dt_ref, what="dt = W_dt (W_x u)[:R]")
    _close(B, s[:, R:R + N], what="B rows of W_x u")
    _close(Cm, s[:, R + N:], what="C rows of W_x u")
    o2, _, h2 = oracle.tree(lay, parents, u, z, dt_ref, s[:, R:R + N], s[:, R + N:], conv0=c0, h0=h0, flags=lay.flags | oracle.PRECONV, _lib_override=L)
    _close(out, o2, what="projection tree: out")
    _close(hn, h2, what="projection tree: state")
    _close(cn, cu_nodes, rtol=0, atol=0, what="projection tree: conv window")


def pin_proj_selectors(L=None):
    """One-hot weights turn the projections into gathers: B[n] = u[n], C[n] = u[N+n], dt[d] = u[(d + 1) % R']."""
    lay, _, _, parents, x, z, c0, h0 = _proj_problem(21, Dn=8, N=3, R=4)
    Dn, N, W = lay.dims
    R = 4
    Wx = np.zeros((R + 2 * N, Dn)); Wdt = np.zeros((Dn, R))
    for r in range(R): Wx[r, 7 - r] = 1.0                  # s[r] = u[7 - r]
    for n in range(N): Wx[R + n, n] = 1.0; Wx[R + N + n, N + n] = 1.0
    for d in range(Dn): Wdt[d, (d + 1) % R] = 1.0          # dt[d] = s[(d+1) % R] = u[7 - (d+1) % R]
    out, _, hn, dt, B, Cm = oracle.tree_proj(lay, Wx, Wdt, parents, x, z, conv0=c0, h0=h0, _lib_override=L)
    zero = np.zeros_like(x); zbc = np.zeros((len(parents), N))
    u, _, _ = oracle.tree(lay, parents, x, zero, zero, zbc, zbc, conv0=c0, h0=h0, flags=lay.flags | oracle.CONV_ONLY, _lib_override=L)
    _close(B, u[:, :N], rtol=0, atol=0, what="B gathers u[0:N]")
    _close(Cm, u[:, N:2 * N], rtol=0, atol=0, what="C gathers u[N:2N]")
    dsel = np.stack([u[:, 7 - (d + 1) % R] for d in range(Dn)], axis=1)
    _close(dt, dsel, rtol=0, atol=0, what="dt gathers through both projections")
    o2, _, h2 = oracle.tree(lay, parents, u, z, dsel, u[:, :N], u[:, N:2 * N], conv0=c0, h0=h0, flags=lay.flags | oracle.PRECONV, _lib_override=L)
    _close(out, o2, rtol=0, atol=0, what="selector tree: out")
    _close(hn, h2, rtol=0, atol=0, what="selector tree: state")


def pin_proj_zero_weights(L=None):
    """W_x = 0: dt = 0, B = C = 0, so out = D u SiLU(z) and the state only decays by exp(softplus(dt_bias) A) per step."""
    lay, Wx, Wdt, parents, x, z, c0, h0 = _proj_problem(22)
    Dn, N, W = lay.dims
    out, _, hn, dt, B, Cm = oracle.tree_proj(lay, 0.0 * Wx, Wdt, parents, x, z, conv0=c0, h0=h0, _lib_override=L)
    zero = np.zeros_like(x); zbc = np.zeros((len(parents), N))
    u, _, _ = oracle.tree(lay, parents, x, zero, zero, zbc, zbc, conv0=c0, h0=h0, flags=lay.flags | oracle.CONV_ONLY, _lib_override=L)
    _close(dt, zero, rtol=0, atol=0, what="zero W_x: dt"); _close(B, zbc, rtol=0, atol=0, what="zero W_x: B")
    silu = np.vectorize(lambda v: v / (1.0 + math.exp(-v)))
    _close(out, lay.D[None, :] * u * silu(z), what="zero W_x: out")
    delta = np.array([math.log1p(math.exp(b)) for b in lay.dt_bias])
    depth = np.zeros(len(parents), dtype=int)
    for v in range(1, len(parents)): depth[v] = depth[parents[v]] + 1
    for v in range(len(parents)):
        _close(hn[v], np.exp(delta[:, None] * lay.A * (depth[v] + 1)) * h0, what=f"zero W_x: state of node {v}")


# ------------------------------------------------------------------ Mamba-2 (SSD): one scalar A per head
def _ssd_problem(i, H=3, P=2, N=5, W=4, T=19, conv_bias=True):
    g = _rng(i)
    Dn = H * P
    A = -g.uniform(0.3, 4.0, H); Dsk = g.normal(size=Dn); w = g.normal(scale=0.5, size=(Dn, W))
    cb = g.normal(size=Dn) if conv_bias else None
    bias = g.normal(size=H) - 3
    lay = oracle.SsdLayer(A, Dsk, w, cb, bias, P, N, flags=oracle.DT_SOFTPLUS)
    x = g.normal(size=(T, Dn)); z = g.normal(size=(T, Dn)); dt = g.normal(size=(T, H))
    B = g.normal(size=(T, N)); Cm = g.normal(size=(T, N))
    return lay, x, z, dt, B, Cm


def _ssd_as_s6(lay):
    """The S6 layer an SSD layer IS: every head's A copied to the N states of its P channels, its step-size bias to
    its channels.  (Built here with numpy; nothing of the SSD routine is involved.)"""
    Dn, H, N, W = lay.dims
    A6 = np.repeat(lay.A, lay.headdim)[:, None] * np.ones((1, N))
    bias6 = None if lay.dt_bias is None else np.repeat(lay.dt_bias, lay.headdim)
    return oracle.Layer(A6, lay.D, lay.conv_w, lay.conv_b, bias6, flags=lay.flags)


def pin_ssd_is_s6_with_head_constant_A(L=None):
    """An SSD layer is an S6 layer whose A is constant over the states and over the channels of a head, and whose step
    size is shared by the channels of a head: prefill and tree must agree with mdo_prefill / mdo_tree (pinned above)
    on the expanded constants and the expanded dt, including one-channel heads (P = 1)."""
    for i, (H, P) in enumerate(((3, 2), (4, 1), (1, 5))):
        lay, x, z, dt, B, Cm = _ssd_problem(30 + i, H=H, P=P)
        g = _rng(40 + i)
        Dn, _, N, W = lay.dims
        cu = np.array([0, 3, 4, 19], dtype=np.int32)
        ci = g.normal(size=(3, W - 1, Dn)); hi = g.normal(size=(3, Dn, N))
        got = oracle.ssd_prefill(lay, x, z, dt, B, Cm, cu_seqlens=cu, conv_init=ci, h_init=hi, _lib_override=L)
        want = oracle.prefill(_ssd_as_s6(lay), x, z, np.repeat(dt, P, axis=1), B, Cm, cu_seqlens=cu, conv_init=ci, h_init=hi, _lib_override=L)
        for a, b, nm in zip(got, want, ("out", "window", "state")):
            _close(a, b, what=f"SSD prefill == S6 prefill on expanded constants (H={H}, P={P}): {nm}")
        parents = np.array([-1, 0, 0, 1, 1, 2, 4, 4])
        M = len(parents)
        got = oracle.ssd_tree(lay, parents, x[:M], z[:M], dt[:M], B[:M], Cm[:M], conv0=ci[0], h0=hi[0], _lib_override=L)
        want = oracle.tree(_ssd_as_s6(lay), parents, x[:M], z[:M], np.repeat(dt[:M], P, axis=1), B[:M], Cm[:M], conv0=ci[0], h0=hi[0], _lib_override=L)
        for a, b, nm in zip(got, want, ("out", "window", "state")):
            _close(a, b, what=f"SSD tree == S6 tree on expanded constants (H={H}, P={P}): {nm}")


def pin_ssd_geometric_series(L=None):
    """Constant Delta, B, C, u per head and a given h0: h_t = a^t h0 + b (1 - a^t) / (1 - a) with the head's scalar
    a = exp(Delta A), b = Delta B u; A = 0 in one head gives the running sum there."""
    g = _rng(50)
    H, P, N, T, W = 3, 2, 4, 33, 4
    Dn = H * P
    A = -g.uniform(0.2, 3.0, H); A[1] = 0.0
    Dsk = g.normal(size=Dn)
    delta = g.uniform(0.01, 0.3, H)
    u = g.normal(size=Dn); Bc = g.normal(size=N); Cc = g.normal(size=N)
    h0 = g.normal(size=(1, Dn, N))
    lay = oracle.SsdLayer(A, Dsk, _identity_conv(Dn, W), None, None, P, N, flags=oracle.PRECONV)
    out, _, hT = oracle.ssd_prefill(lay, np.tile(u, (T, 1)), np.full((T, Dn), BIG_Z), np.tile(delta, (T, 1)), np.tile(Bc, (T, 1)), np.tile(Cc, (T, 1)),
                                    h_init=h0, _lib_override=L)
    head = np.arange(Dn) // P
    a = np.exp(delta * A)[head][:, None]                            # (D,1)
    b = (delta[head] * u)[:, None] * Bc[None, :]                   # (D,N)
    t = np.arange(1, T + 1)[:, None, None]
    with np.errstate(invalid="ignore", divide="ignore"):
        series = np.where(a[None] == 1.0, t * np.ones_like(a)[None], (1 - a[None] ** t) / (1 - a[None]))
    h = a[None] ** t * h0 + b[None] * series
    y = (h * Cc[None, None, :]).sum(-1) + Dsk[None, :] * u[None, :]
    _close(out, y * BIG_Z, what="SSD geometric series: out")
    _close(hT[0], h[-1], what="SSD geometric series: final state")


def pin_ssd_head_indexing(L=None):
    """Changing the step size or A of ONE head changes the outputs and states of exactly that head's P channels
    (d = j P + p), and nothing else."""
    lay, x, z, dt, B, Cm = _ssd_problem(60, H=4, P=3)
    base = oracle.ssd_prefill(lay, x, z, dt, B, Cm, _lib_override=L)
    Dn, H, N, W = lay.dims
    P = lay.headdim
    for j in range(H):
        dt2 = dt.copy(); dt2[:, j] += 0.7
        A2 = lay.A.copy(); A2[j] *= 1.5
        for alt in (oracle.ssd_prefill(lay, x, z, dt2, B, Cm, _lib_override=L),
                    oracle.ssd_prefill(oracle.SsdLayer(A2, lay.D, lay.conv_w, lay.conv_b, lay.dt_bias, P, N, flags=lay.flags), x, z, dt, B, Cm, _lib_override=L)):
            moved = np.abs(alt[0] - base[0]).max(axis=0) > 0
            want = (np.arange(Dn) // P) == j
            assert np.array_equal(moved, want), f"head {j}: channels that moved {np.nonzero(moved)[0]}, expected {np.nonzero(want)[0]}"
            smoved = np.abs(alt[2][0] - base[2][0]).max(axis=1) > 0
            assert np.array_equal(smoved, want), f"head {j}: states that moved"


ALL_PINS = [
    pin_scalar_functions, pin_geometric_series, pin_cumulative_sum, pin_frozen_state, pin_brute_force,
    pin_iir_filter, pin_softplus_and_bias_in_path, pin_conv_impulse, pin_conv_numpy,
    pin_conv_feeds_recurrence, pin_prefill_handoff, pin_prefill_equals_chain, pin_tree_paths, pin_varlen,
    pin_proj_library_matmul, pin_proj_selectors, pin_proj_zero_weights,
    pin_ssd_is_s6_with_head_constant_A, pin_ssd_geometric_series, pin_ssd_head_indexing,
]
