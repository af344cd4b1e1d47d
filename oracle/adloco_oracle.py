"""fp64 CPU oracle for the AdLoCo norm test, switch mode and outer step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain restatement of what
the paper defines; the tests compare the CUDA library against it and the
benchmark times it as a CPU baseline.  It shares no code with the CUDA path
and nothing in the product may import it.

Notation follows the paper: a mini-batch holds b samples, g_i is the gradient
of the loss on sample i, the mini-batch gradient is their mean (Eq. 1),
sigma^2_B is the sample variance of the g_i, eta is the norm-test threshold and
b_{k+1} the requested batch size (Section "Norm test").  The outer step is the
last loop of Algorithm 3 (pseudo-gradient average, then OuterOpt).

All arithmetic is float64 (numpy).  Inputs are the very bytes the GPU reads:
float32 arrays, or bfloat16 arrays handed over as uint16 bit patterns, both
widened exactly.

Readings of the paper taken here (each is a parameter where the paper leaves a
choice):
  * Var_{i in B} of a vector is the trace of the sample covariance,
    (1/(b - ddof)) * sum_i ||g_i - gbar||^2, ddof = 1 by default.
  * b_{k+1} = max(1, ceil(stat)); a zero mean gradient gives stat = +inf.
  * b - ddof <= 0 leaves the variance undefined: V = 0, stat = 0, the batch
    stays at max(1, b_cur).  The same holds when a sum is Inf or NaN (flag
    NONFINITE), which is checked first.
  * OuterOpt is SGD with (optionally Nesterov) momentum, no dampening:
    v' = mu v + d, u = d + mu v' (Nesterov) or v' (heavy ball),
    theta' = theta - lr u, with d the mean over the K instances of
    (theta - theta_k).

Pins (tests/test_oracle_pins.py): exact rational brute force on tiny integer
inputs, closed forms (orthonormal gradients, rank-one layer, zero momentum),
the LocalSGD average as a special case of the outer step, a hand-worked dyadic
example, agreement with the library's SGD optimiser, and invariances; every
function in this file has at least one such pin.  Two readings cannot be
settled from the paper's text -- the variance normaliser (ddof) and the
momentum form of OuterOpt: both are parameters here, each value of them is
pinned (ddof 0 and 1 by the closed forms, Nesterov and heavy-ball momentum by
the library optimiser and the hand-worked example), and which one the authors
meant is recorded as a reading in the design notes.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

FLAG_GROW = 1
FLAG_ACCUMULATE = 2
FLAG_UNDEFINED = 4
FLAG_ZERO_MEAN = 8
FLAG_NONFINITE = 16

INT64_MAX = (1 << 63) - 1


# --------------------------------------------------------------------------
# exact widening of the storage types
# --------------------------------------------------------------------------
def widen(a) -> np.ndarray:
    """float32 / float64 array, or bfloat16 given as uint16 (or int16) bit
    patterns -> float64, exactly."""
    a = np.asarray(a)
    if a.dtype in (np.uint16, np.int16):
        bits = a.view(np.uint16).astype(np.uint32) << np.uint32(16)
        return bits.view(np.float32).astype(np.float64)
    if a.dtype in (np.float32, np.float64):
        return a.astype(np.float64)
    raise TypeError(f"unsupported storage dtype {a.dtype}")


# --------------------------------------------------------------------------
# batch rule and switch mode (scalars)
# --------------------------------------------------------------------------
@dataclass
class NormTestResult:
    sum_sqnorm: float = 0.0      # Q   = sum_i ||g_i||^2
    mean_sqnorm: float = 0.0     # N   = ||gbar||^2
    variance: float = 0.0        # V   = sigma^2_B
    stat: float = 0.0            # V / (eta^2 N)
    batch_count: int = 0         # b
    b_req: int = 1
    accum_steps: int = 1
    b_micro: int = 1
    flags: int = 0
    per_sample_sqnorm: np.ndarray = field(default_factory=lambda: np.zeros(0))
    grad_sum: np.ndarray | None = None


def switch_plan(b_req: int, b_max: int, switch_n: int):
    """Switch mode (Section "Mode switching"; the first branch of Algorithm 3).

    Accumulate only when the requested batch exceeds switch_n * b_max; then the
    micro-batch is b_max and the number of accumulation steps is
    ceil(b_req / b_max).  Otherwise one step with min(b_req, b_max) samples.
    Returns (accumulate?, accum_steps, b_micro).
    """
    if b_req > switch_n * b_max:
        return True, -(-b_req // b_max), b_max
    return False, 1, min(b_req, b_max)


def decide(sum_sqnorm: float, mean_sqnorm: float, variance: float, b: int, *,
           eta: float, ddof: int = 1, b_cur: int = 1, b_max: int = 1,
           b_cap: int = 0, switch_n: int = 2) -> NormTestResult:
    """Batch rule of the approximate norm test:
    b_{k+1} = ceil( sigma^2_B / (eta^2 ||grad F_B||^2) ), then the switch plan."""
    if not (eta > 0.0 and math.isfinite(eta)):
        raise ValueError("eta must be positive and finite")
    r = NormTestResult(sum_sqnorm=sum_sqnorm, mean_sqnorm=mean_sqnorm, batch_count=b)
    if not (math.isfinite(sum_sqnorm) and math.isfinite(mean_sqnorm) and math.isfinite(variance)):
        # an Inf or NaN gradient entry leaves no statistic to test: the batch stays
        r.flags |= FLAG_NONFINITE
        r.variance, r.stat = 0.0, 0.0
        r.b_req = max(1, b_cur)
    elif b - ddof <= 0:
        r.flags |= FLAG_UNDEFINED
        r.variance, r.stat = 0.0, 0.0
        r.b_req = max(1, b_cur)
    elif mean_sqnorm == 0.0:
        r.flags |= FLAG_ZERO_MEAN
        r.variance = variance
        r.stat = math.inf
        r.b_req = b_cap if b_cap > 0 else INT64_MAX
    else:
        r.variance = variance
        r.stat = variance / (eta * eta * mean_sqnorm)
        r.b_req = max(1, math.ceil(r.stat)) if r.stat < 9.0e18 else INT64_MAX
    if b_cap > 0:
        r.b_req = min(r.b_req, b_cap)
    if r.b_req > b_cur:
        r.flags |= FLAG_GROW
    acc, r.accum_steps, r.b_micro = switch_plan(r.b_req, b_max, switch_n)
    if acc:
        r.flags |= FLAG_ACCUMULATE
    return r


# --------------------------------------------------------------------------
# norm test on materialised per-sample gradients
# --------------------------------------------------------------------------
def norm_test(G, *, eta: float, ddof: int = 1, b_cur: int = 1, b_max: int = 1,
              b_cap: int = 0, switch_n: int = 2, want_sum: bool = False) -> NormTestResult:
    """Norm test on G [b, P], row i = g_i.

    gbar = (1/b) sum_i g_i                       (Eq. 1)
    n_i  = ||g_i||^2
    N    = ||gbar||^2
    V    = (1/(b-ddof)) sum_i ||g_i - gbar||^2   (sample variance, two passes)
    stat = V / (eta^2 N);  b_{k+1} = ceil(stat)  (Section "Norm test")
    """
    G = np.asarray(G)
    b, P = G.shape
    total = np.zeros(P, dtype=np.float64)
    for i in range(b):
        total += widen(G[i])
    gbar = total / b
    n = np.zeros(b, dtype=np.float64)
    dev = 0.0
    for i in range(b):
        g = widen(G[i])
        n[i] = float(np.dot(g, g))
        c = g - gbar
        dev += float(np.dot(c, c))
    N = float(np.dot(gbar, gbar))
    V = dev / (b - ddof) if b - ddof > 0 else 0.0
    r = decide(float(n.sum()), N, V, b, eta=eta, ddof=ddof, b_cur=b_cur,
               b_max=b_max, b_cap=b_cap, switch_n=switch_n)
    r.per_sample_sqnorm = n
    if want_sum:
        r.grad_sum = total
    return r


# --------------------------------------------------------------------------
# inner-product test and augmented inner-product test
# --------------------------------------------------------------------------
@dataclass
class InnerProductResult:
    var_ip: float = 0.0        # Var_i <g_i, gbar>
    stat_ip: float = 0.0       # var_ip / (theta^2 ||gbar||^4)
    var_orth: float = 0.0      # Var_i of the component of g_i orthogonal to gbar
    stat_orth: float = 0.0     # var_orth / (nu^2 ||gbar||^2)
    mean_sqnorm: float = 0.0
    batch_count: int = 0
    b_ip: int = 1
    b_aug: int = 1
    flags: int = 0
    inner_products: np.ndarray = field(default_factory=lambda: np.zeros(0))


def inner_product_tests(G, *, theta: float, nu: float, ddof: int = 1, b_cur: int = 1,
                        b_cap: int = 0) -> InnerProductResult:
    """Inner-product test and its augmented form (Section "Inner product test").

    p_i      = <g_i, gbar>
    b_ip     = ceil( Var_i(p_i) / (theta^2 ||gbar||^4) )
    o_i      = g_i - (p_i / ||gbar||^2) gbar            (component orthogonal to gbar)
    b_aug    = ceil( max{ b_ip, Var_i(o_i) / (nu^2 ||gbar||^2) } )
    Variances use the (b - ddof) normaliser; the variance of the vectors o_i is
    the trace of their sample covariance, as for the norm test.
    """
    if not (theta > 0.0 and math.isfinite(theta) and nu > 0.0 and math.isfinite(nu)):
        raise ValueError("theta and nu must be positive and finite")
    G = np.asarray(G)
    b, P = G.shape
    total = np.zeros(P, dtype=np.float64)
    for i in range(b):
        total += widen(G[i])
    gbar = total / b
    N = float(np.dot(gbar, gbar))
    r = InnerProductResult(mean_sqnorm=N, batch_count=b)
    if not math.isfinite(N):
        r.flags |= FLAG_NONFINITE
        r.b_ip = r.b_aug = max(1, b_cur)
    elif b - ddof <= 0:
        r.flags |= FLAG_UNDEFINED
        r.b_ip = r.b_aug = max(1, b_cur)
    elif N == 0.0:
        r.flags |= FLAG_ZERO_MEAN
        r.stat_ip = r.stat_orth = math.inf
        r.b_ip = r.b_aug = b_cap if b_cap > 0 else INT64_MAX
    else:
        p = np.zeros(b, dtype=np.float64)
        for i in range(b):
            p[i] = float(np.dot(widen(G[i]), gbar))
        pbar = float(p.sum()) / b
        r.var_ip = float(((p - pbar) ** 2).sum()) / (b - ddof)
        r.stat_ip = r.var_ip / (theta * theta * N * N)
        obar = np.zeros(P, dtype=np.float64)
        for i in range(b):
            obar += widen(G[i]) - (p[i] / N) * gbar
        obar /= b
        dev = 0.0
        for i in range(b):
            c = widen(G[i]) - (p[i] / N) * gbar - obar
            dev += float(np.dot(c, c))
        r.var_orth = dev / (b - ddof)
        r.stat_orth = r.var_orth / (nu * nu * N)
        r.b_ip = max(1, math.ceil(r.stat_ip)) if r.stat_ip < 9.0e18 else INT64_MAX
        b_orth = max(1, math.ceil(r.stat_orth)) if r.stat_orth < 9.0e18 else INT64_MAX
        r.b_aug = max(r.b_ip, b_orth)
        r.inner_products = p
    if b_cap > 0:
        r.b_ip, r.b_aug = min(r.b_ip, b_cap), min(r.b_aug, b_cap)
    if r.b_aug > b_cur:
        r.flags |= FLAG_GROW
    return r


# --------------------------------------------------------------------------
# linear layers: per-sample weight gradients from activations and output grads
# --------------------------------------------------------------------------
def per_sample_weight_grad(X_i, D_i) -> np.ndarray:
    """Weight gradient of one sample of a linear layer y = W x:
    G_i = sum_t delta_t x_t^T = D_i^T X_i  ([d_out, d_in]), tokens t of the
    sample's sequence; X_i [T, d_in], D_i [T, d_out]."""
    return widen(D_i).T @ widen(X_i)


def linear_layer_terms(X, D):
    """For one linear layer and a batch: n_i = ||G_i||_F^2 for every sample and
    S = sum_i G_i, with G_i formed explicitly (no Gram shortcut)."""
    B = X.shape[0]
    n = np.zeros(B, dtype=np.float64)
    S = np.zeros((D.shape[2], X.shape[2]), dtype=np.float64)
    for i in range(B):
        G_i = per_sample_weight_grad(X[i], D[i])
        n[i] = float(np.sum(G_i * G_i))
        S += G_i
    return n, S


def vector_param_terms(D, X=None):
    """Per-sample gradients of a vector parameter of width d applied at every token:
    a bias (y_t = ... + beta: g_i = sum_t delta_t) or an elementwise gain such as
    LayerNorm's (y_t = gamma * xhat_t: g_i = sum_t delta_t * xhat_t, X = xhat).
    D [B, T, d] (and X [B, T, d]).  Returns n_i = ||g_i||^2 and S = sum_i g_i."""
    B = D.shape[0]
    n = np.zeros(B, dtype=np.float64)
    S = np.zeros(D.shape[2], dtype=np.float64)
    for i in range(B):
        d = widen(D[i])
        g = (d * widen(X[i])).sum(axis=0) if X is not None else d.sum(axis=0)
        n[i] = float(np.dot(g, g))
        S += g
    return n, S


def embedding_terms(ids, D, V: int):
    """Per-sample gradients of an embedding table E [V, d] looked up at every token:
    row v of sample i's gradient is the sum of delta_{i,t} over the tokens t with
    ids[i, t] = v.  ids [B, T] integers, D [B, T, d].  A token whose id lies
    outside [0, V) (padding, an ignore marker) looks up no row of E, so it has no
    term in any row's sum: it is dropped.
    Returns n_i = ||G_i||_F^2 and S = sum_i G_i ([V, d])."""
    ids = np.asarray(ids)
    B = ids.shape[0]
    d = D.shape[2]
    n = np.zeros(B, dtype=np.float64)
    S = np.zeros((V, d), dtype=np.float64)
    for i in range(B):
        G_i = np.zeros((V, d), dtype=np.float64)
        inside = (ids[i] >= 0) & (ids[i] < V)
        np.add.at(G_i, ids[i][inside], widen(D[i])[inside])
        n[i] = float(np.sum(G_i * G_i))
        S += G_i
    return n, S


def linear_layers_norm_test(layers, *, eta: float, ddof: int = 1, b_cur: int = 1,
                            b_max: int = 1, b_cap: int = 0, switch_n: int = 2,
                            two_pass: bool = True) -> NormTestResult:
    """Norm test over the weights of several linear layers; `layers` is a list
    of (X [B,T,d_in], D [B,T,d_out]).  A sample's gradient is the concatenation
    of its per-layer weight gradients.

    two_pass=True materialises every G_i and applies `norm_test`'s definition
    to the flattened [B, P_total] matrix.  two_pass=False (for sizes whose
    per-sample gradients do not fit in memory) uses
    sum_i ||g_i - gbar||^2 = sum_i n_i - b ||gbar||^2.
    """
    B = layers[0][0].shape[0]
    if two_pass:
        flat = [np.stack([per_sample_weight_grad(X[i], D[i]).ravel() for i in range(B)])
                for X, D in layers]
        G = np.concatenate(flat, axis=1)
        return norm_test(G, eta=eta, ddof=ddof, b_cur=b_cur, b_max=b_max, b_cap=b_cap,
                         switch_n=switch_n, want_sum=True)
    n = np.zeros(B, dtype=np.float64)
    sums = []
    for X, D in layers:
        n_l, S_l = linear_layer_terms(X, D)
        n += n_l
        sums.append(S_l)
    return norm_test_from_sums(n, sums, B, eta=eta, ddof=ddof, b_cur=b_cur, b_max=b_max,
                          b_cap=b_cap, switch_n=switch_n)


def norm_test_from_sums(n, sums, b: int, *, eta: float, ddof: int = 1, b_cur: int = 1,
                   b_max: int = 1, b_cap: int = 0, switch_n: int = 2) -> NormTestResult:
    """The test from Q = sum_i n_i and the gradient sums S (one array per
    parameter buffer): N = ||S/b||^2, V = (Q - b N)/(b - ddof)."""
    n = np.asarray(n, dtype=np.float64)
    Q = float(n.sum())
    N = 0.0
    for S in sums:
        m = np.asarray(S, dtype=np.float64).ravel() / b
        N += float(np.dot(m, m))
    V = (Q - b * N) / (b - ddof) if b - ddof > 0 else 0.0
    r = decide(Q, N, V, b, eta=eta, ddof=ddof, b_cur=b_cur, b_max=b_max,
               b_cap=b_cap, switch_n=switch_n)
    r.per_sample_sqnorm = n
    r.grad_sum = sums
    return r


# --------------------------------------------------------------------------
# switch-mode accumulation of the test sums
# --------------------------------------------------------------------------
def accumulated_norm_test(micro_batches, **params) -> NormTestResult:
    """Switch mode processes a batch that exceeds b_max as `accum` micro-batches
    (first branch of Algorithm 3: g <- g + grad L(x; B) per micro-batch).  The
    test on the accumulated batch is, by definition, the one-shot norm test on
    the concatenation of the micro-batches."""
    return norm_test(np.concatenate([np.asarray(m) for m in micro_batches], axis=0), **params)


def accumulated_norm_test_by_sums(micro_batches, *, eta: float, ddof: int = 1, **kw) -> NormTestResult:
    """The same test taken the way the accumulation proceeds: per micro-batch
    add Q += sum_i ||g_i||^2 and S += sum_i g_i, then one test from (Q, S, b)."""
    Q_terms = []
    S = None
    b = 0
    for m in micro_batches:
        m = np.asarray(m)
        for i in range(m.shape[0]):
            g = widen(m[i])
            Q_terms.append(float(np.dot(g, g)))
            S = g.copy() if S is None else S + g
        b += m.shape[0]
    return norm_test_from_sums(Q_terms, [S], b, eta=eta, ddof=ddof, **kw)


# --------------------------------------------------------------------------
# outer step
# --------------------------------------------------------------------------
def outer_step(theta, instances, mom, *, lr: float, momentum: float, nesterov: bool = True):
    """One outer step for one trainer (last loop of Algorithm 3).

    d      = (1/K) sum_k (theta - theta_k)        pseudo-gradient average
    v'     = momentum * v + d
    u      = d + momentum * v'  (Nesterov)  |  v'  (heavy ball)
    theta' = theta - lr * u                       OuterOpt
    Returns (theta', v') in float64.
    """
    th = widen(theta)
    v = widen(mom)
    K = len(instances)
    acc = np.zeros_like(th)
    for k in range(K):
        acc += th - widen(instances[k])
    d = acc / K
    v_new = momentum * v + d
    u = d + momentum * v_new if nesterov else v_new
    return th - lr * u, v_new


# --------------------------------------------------------------------------
# trainer merge (Algorithms 1 and 2)
# --------------------------------------------------------------------------
def check_merge(b_req, w: int):
    """CheckMerge (Algorithm 1): indices of the w trainers with the smallest
    requested batch; empty when w = 0, there is at most one trainer, or w
    exceeds the number of trainers.  Ties keep the lower index first."""
    k = len(b_req)
    if w == 0 or k <= 1:
        return []
    order = sorted(range(k), key=lambda i: (b_req[i], i))
    return order[:w] if w <= k else []


def do_merge(params, b_req):
    """DoMerge (Algorithm 2): x_merge = sum_j b_j x_j / sum_j b_j over the merge
    set; the representative is the member with the largest b_req (lowest index
    on ties).  Returns (x_merge float64, index of the representative)."""
    w_sum = float(sum(b_req))
    x = np.zeros_like(widen(params[0]))
    for p, b in zip(params, b_req):
        x += float(b) * widen(p)
    rep = max(range(len(b_req)), key=lambda j: (b_req[j], -j))
    return x / w_sum, rep
