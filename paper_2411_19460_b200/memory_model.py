"""Memory model of Multi-Axis Gradient Checkpointing and the choice of the two intervals.

Host-side arithmetic only (no device work): Eq. 4 (unit-cost model), its critical point (Eq. 5-7), the two
boundary cases with their AM-GM lower bounds (Eq. 8-9), the regimes of Eq. 10, and the estimator of
Appendix C, M = M_L + M_S + M_grid + M_state, with per-model constants in bf16-element units.

`L` is the number of layers, `S` the sequence length, `l` and `s` the checkpoint intervals along the two
axes, as in the paper.
"""
from dataclasses import dataclass
import math


# ------------------------------------------------------------------ Eq. 4-11: the unit-cost model
def unit_memory(L, S, l, s):
    """Eq. 4: layer-axis checkpoints + sequence-axis checkpoints + one grid cell."""
    return L * S / l + L * S / s + l * s


def critical_point(L, S):
    """Eq. 5-7: the stationary point l = s = (L S)^(1/3) and the memory there, 3 (L S)^(2/3)."""
    c = (L * S) ** (1.0 / 3.0)
    return c, c, 3.0 * (L * S) ** (2.0 / 3.0)


def l_bound_memory(L, S, s):
    """Eq. 8, left side: the edge l = L (no layer-axis recomputation split)."""
    return S + L * (S / s + s)


def s_bound_memory(L, S, l):
    """Eq. 9, left side: the edge s = S."""
    return L + S * (L / l + l)


def l_bound_floor(L, S):
    """Eq. 8, right side (AM-GM, reached at s = sqrt(S))."""
    return S + 2.0 * L * math.sqrt(S)


def s_bound_floor(L, S):
    """Eq. 9, right side (AM-GM, reached at l = sqrt(L))."""
    return L + 2.0 * S * math.sqrt(L)


def regime(L, S):
    """Eq. 10: which term sets the optimum.  'interior' when the stationary point lies inside
    1 <= l <= L, 1 <= s <= S (L <= S^2 and S <= L^2), 'S' when L^2 <= S, 'L' when S^2 <= L."""
    if L * L <= S:
        return "S"
    if S * S <= L:
        return "L"
    return "interior"


# ------------------------------------------------------------------ Appendix C: the estimator
@dataclass(frozen=True)
class MemoryConstants:
    """Per-model constants, in elements of `bytes_per_element` bytes (an fp32 value counts as two bf16
    elements).  c_l: per token and checkpointed layer; c_s: per layer and checkpointed position;
    c_grid: per token and layer inside the cell being restored; c_state: per token of the segment whose
    states the layer kernel rebuilds in its backward."""
    c_l: float
    c_s: float
    c_grid: float
    c_state: float
    bytes_per_element: int = 2


def mamba2_constants(d_model, *, expand=2, headdim=64, d_state=128, ngroups=1, d_conv=4):
    """The constants of Appendix C's table from the dimensions of a Mamba-2 block.
    c_l     = d_model                                   (the block input)
    c_s     = H P N + (d_conv-1)(d_inner + 2 G N)       (SSM state + convolution state)
    c_grid  = (2 d_inner + 2 G N + H) + d_inner         (in_proj output + the scan output)
    c_state = H P N + (d_inner + 2 G N)
    """
    d_inner = expand * d_model
    H = d_inner // headdim
    conv_dim = d_inner + 2 * ngroups * d_state
    hpn = H * headdim * d_state
    return MemoryConstants(c_l=d_model, c_s=hpn + (d_conv - 1) * conv_dim,
                           c_grid=(2 * d_inner + 2 * ngroups * d_state + H) + d_inner, c_state=hpn + conv_dim)


@dataclass(frozen=True)
class MemoryEstimate:
    l_ckpt: float
    s_ckpt: float
    grid: float
    state: float

    @property
    def total(self):
        return self.l_ckpt + self.s_ckpt + self.grid + self.state


def expected_memory(L, S, l, s, c):
    """Appendix C: the four terms in bytes."""
    e = c.bytes_per_element
    return MemoryEstimate(l_ckpt=L * S / l * c.c_l * e, s_ckpt=L * S / s * c.c_s * e,
                          grid=l * s * c.c_grid * e, state=s * c.c_state * e)


def continuous_optimum(L, S, c):
    """Stationary point of the Appendix C total over real l, s > 0, clipped to [1,L] x [1,S] per axis:
    dM/dl = 0 gives l = sqrt(L S c_l / (s c_grid)); dM/ds = 0 gives s = sqrt(L S c_s / (l c_grid + c_state)).
    Solved by alternating the two (each step is the exact minimiser along its axis, M is convex along each)."""
    l, s = min(max(math.sqrt(L), 1.0), L), min(max(math.sqrt(S), 1.0), S)
    for _ in range(200):
        l_new = min(max(math.sqrt(L * S * c.c_l / (s * c.c_grid)), 1.0), float(L))
        s_new = min(max(math.sqrt(L * S * c.c_s / (l_new * c.c_grid + c.c_state)), 1.0), float(S))
        if abs(l_new - l) < 1e-12 * l and abs(s_new - s) < 1e-12 * s:
            l, s = l_new, s_new
            break
        l, s = l_new, s_new
    return l, s, expected_memory(L, S, l, s, c).total


def candidate_intervals(L, S, seg_multiple=1):
    """The integer grid the chooser searches: every l in 1..L; every s that is a multiple of
    `seg_multiple` (the layer kernel's chunk length) and divides S."""
    ls = list(range(1, L + 1))
    ss = [s for s in range(seg_multiple, S + 1, seg_multiple) if S % s == 0]
    return ls, ss


def choose_intervals(L, S, c, *, seg_multiple=1, budget_bytes=None):
    """(l, s, estimate): the admissible pair with the least estimated memory; with `budget_bytes`, the
    pair that fits the budget with the least recomputation instead (the smallest l, since a cell of l
    layers re-runs l-1 of them forward, then the largest s), or None when nothing fits."""
    ls, ss = candidate_intervals(L, S, seg_multiple)
    if not ss:
        raise ValueError("no admissible sequence interval")
    best = None
    for l in ls:
        for s in ss:
            est = expected_memory(L, S, l, s, c)
            if budget_bytes is None:
                key = (est.total, l, -s)
            elif est.total <= budget_bytes:
                key = (l, -s, est.total)
            else:
                continue
            if best is None or key < best[0]:
                best = (key, l, s, est)
    return None if best is None else best[1:]


# ------------------------------------------------------------------ this library's own layout
def libssd_constants(H, P, N, G, *, elem_bytes=2):
    """Constants of the SSD-only layer stack driven by `stack.LayerStack`, in elements of `elem_bytes`:
    it keeps the layer input [H,P] per token (c_l), the fp32 state [H,P,N] per layer and segment (c_s);
    a cell holds l-1 recomputed layer inputs per token (c_grid ~ H P per extra layer); the per-segment
    scratch of the kernels is reported by ssd_workspace_bytes and is not modelled here (c_state = 0)."""
    return MemoryConstants(c_l=H * P, c_s=H * P * N * 4 / elem_bytes, c_grid=H * P, c_state=0.0,
                           bytes_per_element=elem_bytes)


def layer_stack_bytes(L, S, l, s, H, P, N, *, elem_bytes=2):
    """Exactly what LayerStack allocates as checkpoints (layer inputs incl. the stack's input and output,
    boundary states incl. the final one), for comparison with its checkpoint_bytes()."""
    kept = 1 + len([j for j in range(1, L + 1) if j % l == 0 or j == L])
    return dict(layer_inputs=kept * S * H * P * elem_bytes, boundary_states=L * (S // s + 1) * H * P * N * 4,
                cell_inputs=(l - 1) * s * H * P * elem_bytes)
