"""Rollout comparison of two environment backends and an equivalence test on
episode returns.

`compare_rollouts` is the paper's Level-3 check (Sec. 3.2, Algorithm 1: matched
seeds, identical action sequences, obs / reward / done compared at every step)
written for any two objects with the batch surface of this package
(`rollout(T, action_mode, actions)`, `get_state()`, `set_state(soa, t)`,
`episode_stats()`): the CUDA handle wrapper, a CPU implementation, or a test
double.  When a call disagrees it rewinds both backends to the state before
the call and replays it one step at a time, so the report names the first
diverging step, env and output component - the localisation that the paper
argues rollout-only checks lack.

`tost_equivalence` is the two one-sided t-tests procedure the paper uses for
its Level-4 cross-backend comparison (equivalence of mean returns within a
margin, alpha = 0.05); `episode_returns` cuts reward / done streams into the
per-episode returns it needs.

Host-side analysis only (numpy); nothing here is on the simulation hot path.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

OBS_NAMES = ("ball_x", "ball_y", "ball_vx", "ball_vy", "agent_paddle_y", "opponent_paddle_y")
STATE_NAMES = ("bx", "by", "vx", "vy", "apy", "opy", "score_a", "score_o", "ep_len", "episode",
               "prev_action")


def _host(x) -> np.ndarray:
    """numpy view of a numpy array or of a (possibly device) torch tensor."""
    if isinstance(x, np.ndarray):
        return x
    return x.detach().cpu().numpy()


@dataclass
class Divergence:
    call: int              # index of the rollout call in the schedule
    step: int              # global agent step t at which the outputs first differ
    env: int               # local env index
    component: str         # e.g. "obs.ball_vy", "reward", "done", "state.apy", "stats"
    value_a: object
    value_b: object
    mismatching_elements: int  # in that component, on that step

    def __str__(self):
        return ("first divergence in call %d at step %d, env %d, %s: %r vs %r (%d elements of that "
                "component differ on this step)" % (self.call, self.step, self.env, self.component,
                                                    self.value_a, self.value_b,
                                                    self.mismatching_elements))


@dataclass
class Report:
    equal: bool
    steps_compared: int = 0
    env_steps_compared: int = 0
    episodes_finished: int = 0
    divergence: Optional[Divergence] = None
    notes: List[str] = field(default_factory=list)

    def __str__(self):
        if self.equal:
            return "equal over %d steps (%d env-steps, %d finished episodes)" % (
                self.steps_compared, self.env_steps_compared, self.episodes_finished)
        return str(self.divergence)


def _first_output_difference(out_a, out_b, pixel: bool):
    """(step index, env, component, va, vb, count) of the first differing output
    element in call order, or None.  Floats are compared by bit pattern."""
    obs_a, rew_a, done_a = (_host(x) for x in out_a)
    obs_b, rew_b, done_b = (_host(x) for x in out_b)
    T = rew_a.shape[0]
    best = None
    if not pixel:
        da = obs_a.view(np.uint32) != obs_b.view(np.uint32)
        if da.any():
            t, n, k = (int(v) for v in np.argwhere(da)[0])
            best = (t, n, "obs." + OBS_NAMES[k], float(obs_a[t, n, k]), float(obs_b[t, n, k]),
                    int(da[t].sum()))
    for name, xa, xb in (("reward", rew_a, rew_b), ("done", done_a, done_b)):
        d = xa.view(np.uint8 if xa.dtype == np.uint8 else np.uint32) != \
            xb.view(np.uint8 if xb.dtype == np.uint8 else np.uint32)
        if d.any():
            t, n = (int(v) for v in np.argwhere(d)[0])
            cand = (t, n, name, xa[t, n].item(), xb[t, n].item(), int(d[t].sum()))
            if best is None or (cand[0], cand[1]) < (best[0], best[1]):
                best = cand
    if pixel and best is None:
        d = obs_a != obs_b
        if d.any():
            n, s, i, j = (int(v) for v in np.argwhere(d)[0])
            best = (T - 1, n, "ring[slot %d][%d][%d]" % (s, i, j), int(obs_a[n, s, i, j]),
                    int(obs_b[n, s, i, j]), int(d.sum()))
    return best


def _state_difference(sa: np.ndarray, sb: np.ndarray):
    d = sa != sb
    if not d.any():
        return None
    # the lowest env first, then field order
    envs = np.argwhere(d.any(axis=0))[:, 0]
    n = int(envs[0])
    f = int(np.argwhere(d[:, n])[0, 0])
    return n, "state." + STATE_NAMES[f], int(sa[f, n]), int(sb[f, n]), int(d.sum())


def compare_rollouts(a, b, schedule: Sequence[Tuple[int, int]],
                     actions_for: Optional[Callable[[int, int], np.ndarray]] = None,
                     pixel: bool = False, localise: bool = True) -> Report:
    """Run the same schedule of rollout calls on backends `a` and `b` and compare
    obs / reward / done of every step, the state after every call and the episode
    statistics.

    schedule:    sequence of (T, action_mode) calls.
    actions_for: for action_mode 2, a function (call_index, T) -> uint8 [T, n]
                 giving the action bytes fed to both backends (a torch device
                 copy is made for a backend whose `device_actions` attribute is
                 true); for action_mode 3, (call_index, T) -> int.
    localise:    on a mismatch, rewind both backends with set_state and replay the
                 call step by step to name the first diverging step.

    Both backends must start from the same state (e.g. both freshly created with
    the same seed)."""
    report = Report(equal=True)

    def feed(backend, mode, acts):
        if mode == 2 and getattr(backend, "device_actions", False):
            import torch
            return torch.from_numpy(np.ascontiguousarray(acts)).cuda()
        return acts

    def run(backend, T, mode, acts):
        if mode in (2, 3):
            return backend.rollout(T, mode, feed(backend, mode, acts))
        return backend.rollout(T, mode)

    for ci, (T, mode) in enumerate(schedule):
        sa0, ta0 = a.get_state()
        sb0, tb0 = b.get_state()
        if ta0 != tb0 or _state_difference(sa0, sb0) is not None:
            sd = _state_difference(sa0, sb0)
            report.equal = False
            report.divergence = Divergence(ci, int(ta0), sd[0] if sd else 0,
                                           sd[1] if sd else "step counter",
                                           sd[2] if sd else ta0, sd[3] if sd else tb0,
                                           sd[4] if sd else 1)
            return report
        acts = actions_for(ci, T) if (mode in (2, 3) and actions_for is not None) else None
        out_a = run(a, T, mode, acts)
        out_b = run(b, T, mode, acts)
        diff = _first_output_difference(out_a, out_b, pixel)
        sa1, _ = a.get_state()
        sb1, _ = b.get_state()
        sdiff = _state_difference(sa1, sb1)
        if diff is None and sdiff is None and a.episode_stats() == b.episode_stats():
            report.steps_compared += T
            report.env_steps_compared += T * sa0.shape[1]
            report.episodes_finished += int(_host(out_a[2]).sum())
            continue
        report.equal = False
        if diff is None:
            if sdiff is not None:
                report.divergence = Divergence(ci, int(ta0) + T, sdiff[0], sdiff[1], sdiff[2],
                                               sdiff[3], sdiff[4])
            else:
                report.divergence = Divergence(ci, int(ta0) + T, 0, "stats", a.episode_stats(),
                                               b.episode_stats(), 1)
            return report
        t_rel, n, comp, va, vb, cnt = diff
        report.divergence = Divergence(ci, int(ta0) + t_rel, n, comp, va, vb, cnt)
        if localise and T > 1 and not pixel:
            # rewind and replay one step at a time: confirms the step and shows
            # whether single-step calls diverge at the same place
            a.set_state(sa0, ta0)
            b.set_state(sb0, tb0)
            for s in range(T):
                step_acts = None
                if mode == 2:
                    step_acts = acts[s:s + 1]
                elif mode == 3:
                    step_acts = acts
                d1 = _first_output_difference(run(a, 1, mode, step_acts),
                                              run(b, 1, mode, step_acts), pixel)
                if d1 is not None:
                    report.notes.append("single-step replay diverges at step %d, env %d, %s"
                                        % (int(ta0) + s, d1[1], d1[2]))
                    break
            else:
                report.notes.append("single-step replay of the call agrees: the difference is "
                                    "specific to the %d-step call" % T)
        return report
    return report


def episode_returns(reward, done, carry: Optional[np.ndarray] = None):
    """Cut reward[T, n] / done[T, n] streams into per-episode returns.

    Returns (returns of the episodes that finished, in step-major order; the
    running partial returns of the unfinished episodes, to pass as `carry` with
    the next chunk)."""
    reward = _host(reward).astype(np.float64)
    done = _host(done).astype(bool)
    T, n = reward.shape
    acc = np.zeros(n, dtype=np.float64) if carry is None else np.array(carry, dtype=np.float64)
    finished: List[float] = []
    for t in range(T):
        acc += reward[t]
        idx = np.nonzero(done[t])[0]
        if len(idx):
            finished.extend(acc[idx].tolist())
            acc[idx] = 0.0
    return np.array(finished, dtype=np.float64), acc


def _student_t_sf(t: float, df: float) -> float:
    """P(T > t) for Student's t with df degrees of freedom (df may be fractional),
    through the regularised incomplete beta function (continued fraction)."""
    if not math.isfinite(t):
        return 0.0 if t > 0 else 1.0
    x = df / (df + t * t)
    p = 0.5 * _betainc(0.5 * df, 0.5, x)
    return p if t > 0 else 1.0 - p


def _betainc(a: float, b: float, x: float) -> float:
    if x <= 0.0:
        return 0.0
    if x >= 1.0:
        return 1.0
    ln_front = (math.lgamma(a + b) - math.lgamma(a) - math.lgamma(b) + a * math.log(x)
                + b * math.log1p(-x))
    if x < (a + 1.0) / (a + b + 2.0):
        return math.exp(ln_front) * _betacf(a, b, x) / a
    return 1.0 - math.exp(ln_front) * _betacf(b, a, 1.0 - x) / b


def _betacf(a: float, b: float, x: float) -> float:
    tiny = 1e-300
    qab, qap, qam = a + b, a + 1.0, a - 1.0
    c, d = 1.0, 1.0 - qab * x / qap
    d = 1.0 / (d if abs(d) > tiny else tiny)
    h = d
    for m in range(1, 500):
        m2 = 2 * m
        aa = m * (b - m) * x / ((qam + m2) * (a + m2))
        d = 1.0 + aa * d
        d = 1.0 / (d if abs(d) > tiny else tiny)
        c = 1.0 + aa / c
        c = c if abs(c) > tiny else tiny
        h *= d * c
        aa = -(a + m) * (qab + m) * x / ((a + m2) * (qap + m2))
        d = 1.0 + aa * d
        d = 1.0 / (d if abs(d) > tiny else tiny)
        c = 1.0 + aa / c
        c = c if abs(c) > tiny else tiny
        delta = d * c
        h *= delta
        if abs(delta - 1.0) < 1e-15:
            break
    return h


@dataclass
class TostResult:
    equivalent: bool
    p_value: float       # the larger of the two one-sided p-values
    p_lower: float       # H0: mean_a - mean_b <= -margin
    p_upper: float       # H0: mean_a - mean_b >= +margin
    difference: float
    std_error: float
    dof: float
    margin: float
    alpha: float


def tost_equivalence(xa, xb, margin: float, alpha: float = 0.05) -> TostResult:
    """Two one-sided Welch t-tests: the means of the samples are declared
    equivalent when both `mean_a - mean_b <= -margin` and `>= +margin` are rejected
    at level alpha.  Identical constant samples (zero variance, zero difference)
    are equivalent for any positive margin."""
    xa = np.asarray(xa, dtype=np.float64).ravel()
    xb = np.asarray(xb, dtype=np.float64).ravel()
    if len(xa) < 2 or len(xb) < 2:
        raise ValueError("need at least two observations per sample")
    if margin <= 0:
        raise ValueError("margin must be positive")
    va, vb = xa.var(ddof=1) / len(xa), xb.var(ddof=1) / len(xb)
    diff = float(xa.mean() - xb.mean())
    se2 = va + vb
    if se2 == 0.0:
        inside = abs(diff) < margin
        p = 0.0 if inside else 1.0
        return TostResult(inside, p, p, p, diff, 0.0, float("inf"), margin, alpha)
    se = math.sqrt(se2)
    dof = se2 * se2 / (va * va / (len(xa) - 1) + vb * vb / (len(xb) - 1))
    p_lower = _student_t_sf((diff + margin) / se, dof)      # reject if diff is well above -margin
    p_upper = 1.0 - _student_t_sf((diff - margin) / se, dof)  # reject if diff is well below +margin
    p = max(p_lower, p_upper)
    return TostResult(p < alpha, p, p_lower, p_upper, diff, se, dof, margin, alpha)
