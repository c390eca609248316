"""Placement search on top of the batched placement-cost kernel (the paper's Section VI, Algorithm 1).

What follows the paper: the cost model (Eq. 1-4: a layer's latency is the straggler's computation plus the
straggler's communication), the LP relaxation of the placement problem with the max operators linearised by
auxiliary variables (Eq. 6), and the binary search over the latency budget beta that Algorithm 1 wraps around
the feasibility LP.  What does not: the profiled latency functions f_comp / f_comm are not published, so affine
stand-ins are used (declared in `LatencyModel`); and the rounding: the paper's iterative randomized rounding is
here (`iterative_rounding`, with the constants the paper leaves open declared in `RoundingParams`), but at a vertex
of the LP nearly every latency constraint is tight and its walk can hardly move inside the paper's polytope, so the
search by default uses a deterministic rounding, or on request several randomized roundings that keep only the
assignment and capacity constraints hard, and follows either with a local search.  All candidate batches are
scored on the GPU by `director_placement_cost_batch` - the part of the search that is a data-parallel hot loop.

The LP runs on the host with SciPy (as in the paper's prototype); everything that scores integer placements goes
through an `evaluate(X_batch) -> summary` callable, by default the GPU evaluator below.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class LatencyModel:
    """Affine stand-ins for the paper's profiled latency functions (Section VI-A):
    f_comp(lambda) = comp_fixed + comp_per_token * lambda;  f_comm(D) = comm_per_byte * D (no per-message term).
    bytes_per_token is d of Eq. 3."""
    comp_per_token: float = 1.0
    comp_fixed: float = 0.0
    comm_per_byte: float = 0.0
    bytes_per_token: int = 1

    @property
    def comm_per_token(self) -> float:
        return self.comm_per_byte * self.bytes_per_token

    def latency(self, max_rank_load, max_send_tokens):
        """T_comp + T_comm of one layer (Eq. 2 + Eq. 4) from the two straggler quantities."""
        return self.comp_fixed + self.comp_per_token * np.asarray(max_rank_load, dtype=np.float64) + \
            self.comm_per_token * np.asarray(max_send_tokens, dtype=np.float64)


# ----------------------------------------------------------------------------------------------
# scoring integer placements on the GPU
# ----------------------------------------------------------------------------------------------

class GpuPlacementEvaluator:
    """Scores batches of candidate placements against one workload matrix with director_placement_cost_batch."""

    def __init__(self, director, workload_dev, chunk: int = 8192):
        import torch
        self.torch = torch
        self.d = director
        self.W = workload_dev
        self.R, self.E = workload_dev.shape
        self.chunk = min(chunk, 65535)
        dev = workload_dev.device
        self._load = torch.empty((self.chunk, self.R), dtype=torch.int64, device=dev)
        self._disp = torch.empty((self.chunk, self.R, self.R), dtype=torch.int64, device=dev)
        self._sum = torch.empty((self.chunk, 4), dtype=torch.int64, device=dev)
        self.evaluated = 0

    def __call__(self, X_batch: np.ndarray) -> np.ndarray:
        """X_batch uint8 [n,E,R] -> summary int64 [n,4] = (max load, max send tokens, cross tokens, valid)."""
        torch = self.torch
        X_batch = np.ascontiguousarray(X_batch, dtype=np.uint8)
        out = np.empty((len(X_batch), 4), dtype=np.int64)
        for lo in range(0, len(X_batch), self.chunk):
            xb = torch.from_numpy(X_batch[lo:lo + self.chunk]).to(self.W.device)
            n = xb.shape[0]
            self.d.placement_cost_batch(self.W, n, xb, self._load, self._disp, self._sum)
            out[lo:lo + n] = self._sum[:n].cpu().numpy()
        self.evaluated += len(X_batch)
        return out

    def detail(self, X: np.ndarray):
        """(rank_load [R], dispatch_tokens [R,R]) of one placement."""
        torch = self.torch
        xb = torch.from_numpy(np.ascontiguousarray(X[None], dtype=np.uint8)).to(self.W.device)
        self.d.placement_cost_batch(self.W, 1, xb, self._load, self._disp, self._sum)
        return self._load[0].cpu().numpy(), self._disp[0].cpu().numpy()


# ----------------------------------------------------------------------------------------------
# LP relaxation (Eq. 6) and the binary search of Algorithm 1
# ----------------------------------------------------------------------------------------------

def _lp_matrices(W: np.ndarray, C_max: int, model: LatencyModel):
    """Inequalities A_ub z <= b_ub over z = (x_00..x_{E-1,R-1}, tau_comp, tau_comm) for constraints 6c-6f."""
    R, E = W.shape
    N = W.sum(axis=0).astype(np.float64)
    nx = E * R
    rows, rhs = [], []
    for j in range(R):                                   # 6c: comp_fixed + b_c * sum_i x_ij N_i - tau_comp <= 0
        r = np.zeros(nx + 2)
        r[np.arange(E) * R + j] = model.comp_per_token * N
        r[nx] = -1.0
        rows.append(r)
        rhs.append(-model.comp_fixed)
    for j in range(R):                                   # 6d: sum_{k != j} b_m d sum_i W_ji x_ik - tau_comm <= 0
        r = np.zeros(nx + 2)
        for k in range(R):
            if k != j:
                r[np.arange(E) * R + k] += model.comm_per_token * W[j].astype(np.float64)
        r[nx + 1] = -1.0
        rows.append(r)
        rhs.append(0.0)
    for i in range(E):                                   # 6e: -sum_j x_ij <= -1
        r = np.zeros(nx + 2)
        r[i * R:(i + 1) * R] = -1.0
        rows.append(r)
        rhs.append(-1.0)
    for j in range(R):                                   # 6f: sum_i x_ij <= C_max
        r = np.zeros(nx + 2)
        r[np.arange(E) * R + j] = 1.0
        rows.append(r)
        rhs.append(float(C_max))
    bounds = [(0.0, 1.0)] * nx + [(0.0, None), (0.0, None)]
    return np.array(rows), np.array(rhs), bounds


def lp_minimum(W: np.ndarray, C_max: int, model: LatencyModel):
    """The relaxation solved directly: minimise tau_comp + tau_comm.  Returns (x_bar [E,R], value)."""
    from scipy.optimize import linprog
    R, E = W.shape
    A, b, bounds = _lp_matrices(W, C_max, model)
    c = np.zeros(E * R + 2)
    c[-2:] = 1.0
    res = linprog(c, A_ub=A, b_ub=b, bounds=bounds, method="highs")
    if not res.success:
        raise RuntimeError("LP relaxation failed: " + res.message)
    return res.x[:E * R].reshape(E, R), float(res.fun)


def lp_feasible(W: np.ndarray, C_max: int, model: LatencyModel, beta: float):
    """Feasibility LP of Eq. 6 for a latency budget beta (6b: tau_comp + tau_comm <= beta).
    Returns x_bar [E,R] or None."""
    from scipy.optimize import linprog
    R, E = W.shape
    A, b, bounds = _lp_matrices(W, C_max, model)
    budget = np.zeros(E * R + 2)
    budget[-2:] = 1.0
    res = linprog(np.zeros(E * R + 2), A_ub=np.vstack([A, budget]), b_ub=np.append(b, beta), bounds=bounds,
                  method="highs")
    return res.x[:E * R].reshape(E, R) if res.status == 0 else None


def binary_search_budget(W: np.ndarray, C_max: int, model: LatencyModel, beta_high: float, eps_rel: float = 1e-3,
                         max_steps: int = 40):
    """Algorithm 1's outer loop: bisect the budget beta between 0 and a known feasible value, solving the
    feasibility LP at every step; returns (x_bar_best, beta_best)."""
    lo, hi = 0.0, float(beta_high)
    best = lp_feasible(W, C_max, model, hi)
    if best is None:
        raise RuntimeError("the initial budget is infeasible")
    for _ in range(max_steps):
        if hi - lo <= eps_rel * max(hi, 1e-30):
            break
        mid = 0.5 * (lo + hi)
        x = lp_feasible(W, C_max, model, mid)
        if x is None:
            lo = mid
        else:
            hi, best = mid, x
    return best, hi


# ----------------------------------------------------------------------------------------------
# from the fractional solution to an integer placement
# ----------------------------------------------------------------------------------------------

def round_placement(x_bar: np.ndarray, N: np.ndarray, C_max: int) -> np.ndarray:
    """Deterministic rounding: experts in order of decreasing load take their largest fractional rank that still
    has a free slot (ties: the rank with the smaller load so far, then the lower rank).  Single copy per expert."""
    E, R = x_bar.shape
    X = np.zeros((E, R), dtype=np.uint8)
    free = np.full(R, C_max, dtype=np.int64)
    load = np.zeros(R, dtype=np.int64)
    for e in sorted(range(E), key=lambda i: (-int(N[i]), i)):
        cands = [j for j in range(R) if free[j] > 0]
        j = min(cands, key=lambda j: (-round(float(x_bar[e, j]), 9), int(load[j]), j))
        X[e, j] = 1
        free[j] -= 1
        load[j] += int(N[e])
    return X


# ----------------------------------------------------------------------------------------------
# iterative randomized rounding (Section VI-C, "Iterative Rounding")
# ----------------------------------------------------------------------------------------------

@dataclass(frozen=True)
class RoundingParams:
    """The constants the paper leaves open, as used here: alpha bounds how far a variable may drift inside one
    macro-iteration (distance to its nearest integer at most alpha * scale), gamma is the step size of a micro-step
    in units of the scale, t_micro the number of micro-steps per macro-iteration (None: 40 + 4 * active variables),
    max_macro the number of macro-iterations (None: 4 + 2 * ceil(log2(number of variables)))."""
    alpha: float = 2.0
    gamma: float = 0.25
    t_micro: int | None = None
    max_macro: int | None = None
    tol: float = 1e-6
    # True: the walk also respects the latency constraints 6b-6d for the given budget (the paper's polytope Q).  At a
    # vertex of the LP nearly all of them are tight and the walk can hardly move, so the search uses False: only the
    # assignment and capacity constraints are hard, and the candidates the walk produces are scored afterwards.
    respect_budget: bool = True


def _scales(x: np.ndarray) -> np.ndarray:
    """s_v = 2^-k with dist(x_v, {0,1}) in (2^-(k+1), 2^-k]  (k >= 1 since the distance is at most 1/2; the interval
    is closed on the right, so a distance of exactly 2^-k has scale 2^-k)."""
    d = np.minimum(x, 1.0 - x)
    k = np.floor(-np.log2(np.maximum(d, 1e-300)))
    return 2.0 ** -k


def rounding_potential(x: np.ndarray, scale: np.ndarray) -> float:
    """Phi(x) = sum over fractional v of s_v^-2 * dist(x_v, {0,1})^2."""
    frac = (x > 0.0) & (x < 1.0)
    d = np.minimum(x, 1.0 - x)
    return float(np.sum((d[frac] / scale[frac]) ** 2))


def iterative_rounding(x_bar: np.ndarray, W: np.ndarray, C_max: int, model: LatencyModel, beta: float,
                       rng: np.random.Generator, params: RoundingParams = RoundingParams(), trace: list | None = None):
    """From the fractional LP solution x_bar [E,R] (feasible for budget beta) to an integer placement by the paper's
    constrained random walk:

      macro-iteration: every fractional variable gets the scale s_v = 2^-k of its distance to the nearest integer.
      The walk stays in the polytope Q cut out by (i) the LP's constraints 6b-6g, (ii) dist(x_v, {0,1}) <= alpha s_v
      and (iii) the scale-preserving sums  sum_{v in U_k} x_v = const  over each scale class U_k.  A micro-step draws
      a Gaussian direction with standard deviation s_v per variable, projects it onto the null space of the
      constraints of Q that are tight, and moves by gamma along it (shortened so that no constraint of Q is
      crossed).  A variable that reaches 0 or 1 is clamped there for good.

    Returns (X uint8 [E,R], info).  Variables still fractional after the last macro-iteration are rounded by
    `round_placement`'s rule; the result is repaired to satisfy the assignment and capacity constraints if the
    clamping left it short (info counts both)."""
    R, E = W.shape
    Wf = W.astype(np.float64)
    N = Wf.sum(axis=0)
    tol = params.tol
    x = np.clip(np.array(x_bar, dtype=np.float64), 0.0, 1.0)
    x[x < tol] = 0.0
    x[x > 1.0 - tol] = 1.0
    nx = E * R

    # gradients of the affine pieces of the objective in x (row-major [E,R] flattened): comp_j and comm_j
    G_comp = np.zeros((R, nx))
    G_comm = np.zeros((R, nx))
    for j in range(R):
        G_comp[j, np.arange(E) * R + j] = model.comp_per_token * N
        for k in range(R):
            if k != j:
                G_comm[j, np.arange(E) * R + k] += model.comm_per_token * Wf[j]
    A_assign = np.zeros((E, nx))
    for i in range(E):
        A_assign[i, i * R:(i + 1) * R] = 1.0
    A_cap = np.zeros((R, nx))
    for j in range(R):
        A_cap[j, np.arange(E) * R + j] = 1.0

    n_macro = params.max_macro if params.max_macro is not None else 4 + 2 * int(np.ceil(np.log2(max(nx, 2))))
    info = dict(macro=0, micro=0, clamped=0, fallback=0, repaired=0)
    xf = x.reshape(-1)
    for _ in range(n_macro):
        active = np.flatnonzero((xf > 0.0) & (xf < 1.0))
        if active.size == 0:
            break
        info["macro"] += 1
        scale = np.ones(nx)
        scale[active] = _scales(xf[active])
        classes = np.unique(scale[active])
        A_scale = np.zeros((len(classes), nx))
        for c, sc in enumerate(classes):
            A_scale[c, active[scale[active] == sc]] = 1.0
        frozen = np.zeros(nx, dtype=bool)                  # reached dist = alpha * s_v in this macro-iteration
        if trace is not None:
            trace.append(dict(fractional=int(active.size), potential=rounding_potential(xf, scale)))
        steps = params.t_micro if params.t_micro is not None else 40 + 4 * int(active.size)
        for _ in range(steps):
            mov = active[(xf[active] > 0.0) & (xf[active] < 1.0) & ~frozen[active]]
            if mov.size == 0:
                break
            info["micro"] += 1
            comp = model.comp_fixed + G_comp @ xf
            comm = G_comm @ xf
            budget_slack = beta - (comp.max() + comm.max()) if params.respect_budget else np.inf
            rows = [A_scale]
            s_assign = A_assign @ xf - 1.0
            s_cap = C_max - A_cap @ xf
            rows.append(A_assign[s_assign <= tol])
            rows.append(A_cap[s_cap <= tol])
            scale_tol = tol * max(beta, 1.0)
            if budget_slack <= scale_tol:
                rows.append(G_comp[comp >= comp.max() - scale_tol])
                rows.append(G_comm[comm >= comm.max() - scale_tol])
            r = rng.standard_normal(mov.size) * scale[mov]

            def project(row_blocks):
                A = np.vstack(row_blocks)[:, mov]
                A = A[np.abs(A).sum(axis=1) > 0]
                if not A.shape[0]:
                    return r
                return r - A.T @ np.linalg.lstsq(A @ A.T, A @ r, rcond=None)[0]

            g = project(rows)
            if not np.any(np.abs(g) > 1e-9 * scale[mov]):
                # the tight constraints leave no direction: the scale-preserving sums are a device of the analysis,
                # not of feasibility, so they are the ones to give way
                g = project(rows[1:])
                if not np.any(np.abs(g) > 1e-9 * scale[mov]):
                    break                                   # nothing can move in this macro-iteration any more
            g[np.abs(g) <= 1e-12] = 0.0
            # longest step <= gamma that keeps x inside Q
            t = params.gamma
            pos, neg = g > 1e-14, g < -1e-14
            d = np.minimum(xf[mov], 1.0 - xf[mov])
            toward_int = np.where(xf[mov] <= 0.5, neg, pos)            # moving towards the nearest integer
            away = ~toward_int & (pos | neg)
            lim = np.full(mov.size, np.inf)
            lim[toward_int] = d[toward_int] / np.abs(g[toward_int])                           # reaches 0 or 1
            # bound (ii): the distance grows until x passes 1/2, so it only binds where alpha * s_v < 1/2
            room = np.where(params.alpha * scale[mov] >= 0.5, np.inf, params.alpha * scale[mov] - d)
            lim[away] = np.maximum(room[away], 0.0) / np.abs(g[away])
            t = min(t, float(lim.min()))
            full = np.zeros(nx)
            full[mov] = g
            for Arow, slack in ((A_assign, s_assign), (-A_cap, s_cap)):                        # non-tight 6e, 6f
                rate = -(Arow @ full)
                m = (rate > 1e-9) & (slack > tol)
                if m.any():
                    t = min(t, float((np.maximum(slack[m], 0.0) / rate[m]).min()))
            if budget_slack > scale_tol and params.respect_budget:                             # non-tight 6b-6d
                rate = (G_comp @ full).max() + (G_comm @ full).max()
                if rate > 1e-9:
                    t = min(t, budget_slack / rate)
            if t <= 0.0:
                hit = np.zeros(mov.size, dtype=bool)
                hit[away] = room[away] <= 0.0
                frozen[mov[hit]] = True
                if not hit.any():
                    continue
                continue
            xf[mov] += t * g
            snap0 = xf[mov] <= tol
            snap1 = xf[mov] >= 1.0 - tol
            xf[mov[snap0]] = 0.0
            xf[mov[snap1]] = 1.0
            info["clamped"] += int(snap0.sum() + snap1.sum())
            d2 = np.minimum(xf[mov], 1.0 - xf[mov])
            frozen[mov[(d2 >= params.alpha * scale[mov] - tol) & ~snap0 & ~snap1]] = True
    x = xf.reshape(E, R)
    frac_left = (x > 0.0) & (x < 1.0)
    X = (x >= 1.0 - tol).astype(np.uint8)
    if frac_left.any():                                    # deterministic finish for what the walk left fractional
        info["fallback"] = int(frac_left.sum())
        for i in np.flatnonzero(frac_left.any(axis=1)):
            if X[i].sum() == 0:
                free = np.flatnonzero(X.sum(axis=0) < C_max)
                j = free[np.argmax(x[i, free])] if free.size else int(np.argmax(x[i]))
                X[i, j] = 1
    # repair: every expert hosted, no rank above capacity
    for j in np.flatnonzero(X.sum(axis=0) > C_max):
        hosted = sorted(np.flatnonzero(X[:, j]), key=lambda i: (X[i].sum() < 2, -N[i]))   # drop replicas first
        for i in hosted:
            if X[:, j].sum() <= C_max:
                break
            if X[i].sum() >= 2:
                X[i, j] = 0
                info["repaired"] += 1
        for i in sorted(np.flatnonzero(X[:, j]), key=lambda i: N[i]):
            if X[:, j].sum() <= C_max:
                break
            free = np.flatnonzero(X.sum(axis=0) < C_max)
            X[i, j] = 0
            X[i, free[np.argmin((X[:, free] * N[:, None]).sum(axis=0))]] = 1
            info["repaired"] += 1
    for i in np.flatnonzero(X.sum(axis=1) == 0):
        free = np.flatnonzero(X.sum(axis=0) < C_max)
        X[i, free[np.argmax(x_bar[i, free])]] = 1
        info["repaired"] += 1
    return X, info


def _neighbours(X: np.ndarray, C_max: int):
    """All placements one step away: move one copy of an expert to a rank with a free slot, or swap the copies of
    two experts hosted on different ranks."""
    E, R = X.shape
    used = X.sum(axis=0)
    out = []
    hosts = [np.flatnonzero(X[e]) for e in range(E)]
    for e in range(E):
        for j in hosts[e]:
            for k in range(R):
                if not X[e, k] and used[k] < C_max:
                    Y = X.copy()
                    Y[e, j], Y[e, k] = 0, 1
                    out.append(Y)
    for e in range(E):
        for f in range(e + 1, E):
            for j in hosts[e]:
                for k in hosts[f]:
                    if j != k and not X[e, k] and not X[f, j]:
                        Y = X.copy()
                        Y[e, j], Y[e, k], Y[f, k], Y[f, j] = 0, 1, 0, 1
                        out.append(Y)
    return out


def _replica_additions(X: np.ndarray, C_max: int):
    E, R = X.shape
    used = X.sum(axis=0)
    out = []
    for e in range(E):
        for k in range(R):
            if not X[e, k] and used[k] < C_max:
                Y = X.copy()
                Y[e, k] = 1
                out.append(Y)
    return out


def local_search(evaluate, X0: np.ndarray, C_max: int, model: LatencyModel, allow_replicas: bool = False,
                 max_rounds: int = 200):
    """Steepest descent over the neighbourhood of `_neighbours` (and, if allowed, adding a replica in a free slot);
    every round scores the whole neighbourhood in one batch.  Returns (X, latency, rounds)."""
    X = np.array(X0, dtype=np.uint8)
    s = evaluate(X[None])[0]
    assert s[3] == 1, "the starting placement is invalid"
    cur = float(model.latency(s[0], s[1]))
    rounds = 0
    for rounds in range(1, max_rounds + 1):
        cands = _neighbours(X, C_max) + (_replica_additions(X, C_max) if allow_replicas else [])
        if not cands:
            break
        S = evaluate(np.stack(cands))
        lat = np.where(S[:, 3] == 1, model.latency(S[:, 0], S[:, 1]), np.inf)
        b = int(np.argmin(lat))
        if not lat[b] < cur * (1.0 - 1e-12):
            break
        X, cur = cands[b], float(lat[b])
    return X, cur, rounds


def optimize_placement(W: np.ndarray, C_max: int, model: LatencyModel, evaluate, allow_replicas: bool = False,
                       use_binary_search: bool = True, rounding: str = "deterministic", n_roundings: int = 16,
                       seed: int = 0):
    """Algorithm 1 with the stand-ins described in the module header.  W: int64 [R,E] workload matrix.
    rounding: "deterministic" (round_placement) or "randomized": n_roundings runs of the paper's iterative randomized
    rounding (assignment and capacity hard, latency scored afterwards) plus the deterministic one, all scored in one
    batch, the best one kept.  Either is followed by the local search.
    Returns dict(X, latency, lp_bound, x_bar, rounds, start_latency)."""
    R, E = W.shape
    N = W.sum(axis=0)
    # a feasible starting budget: round-robin placement of the experts in order of load
    X_rr = np.zeros((E, R), dtype=np.uint8)
    for pos, e in enumerate(sorted(range(E), key=lambda i: (-int(N[i]), i))):
        X_rr[e, pos % R] = 1
    s = evaluate(X_rr[None])[0]
    beta_high = float(model.latency(s[0], s[1]))
    if use_binary_search:
        x_bar, bound = binary_search_budget(W, C_max, model, beta_high * (1.0 + 1e-9))
    else:
        x_bar, bound = lp_minimum(W, C_max, model)
    starts = [round_placement(x_bar, N, C_max)]
    if rounding == "randomized":
        rng = np.random.default_rng(seed)
        soft = RoundingParams(respect_budget=False)
        starts += [iterative_rounding(x_bar, W, C_max, model, bound, rng, soft)[0] for _ in range(n_roundings)]
    elif rounding != "deterministic":
        raise ValueError(rounding)
    S = evaluate(np.stack(starts))
    lat0 = np.where(S[:, 3] == 1, model.latency(S[:, 0], S[:, 1]), np.inf)
    b = int(np.argmin(lat0))
    X0, start = starts[b], float(lat0[b])
    if not start <= beta_high:
        X0, start = X_rr, beta_high                      # rounding never has to be worse than the trivial start
    X, lat, rounds = local_search(evaluate, X0, C_max, model, allow_replicas)
    return dict(X=X, latency=lat, lp_bound=bound, x_bar=x_bar, rounds=rounds, start_latency=start)


def enumerate_single_copy(E: int, R: int, C_max: int):
    """Every single-copy placement with at most C_max experts per rank, as uint8 [n,E,R] (tiny E only)."""
    out = []
    assign = [0] * E
    count = [0] * R

    def rec(e):
        if e == E:
            X = np.zeros((E, R), dtype=np.uint8)
            X[np.arange(E), assign] = 1
            out.append(X)
            return
        for j in range(R):
            if count[j] < C_max:
                assign[e] = j
                count[j] += 1
                rec(e + 1)
                count[j] -= 1

    rec(0)
    return np.stack(out)
