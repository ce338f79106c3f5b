"""Closed forms of the paper's analytical cost model, for use with measured attention-stage
bandwidth (host-side arithmetic only; nothing here runs on the GPU).

Notation follows Section 3.1 ("Analytical Setup"): a GPU type has unit-time cost c, memory
bandwidth beta, memory capacity M and peak compute F; alpha = c / beta is the cost per byte of
memory traffic and gamma = c / F the cost per FLOP; m_kv(s) is the KV-cache memory per request
at sequence length s, P_act the GEMM-side parameters activated per request, M_weights the
resident weight footprint.  Units are the caller's choice as long as they are consistent
(the helpers below use bytes, bytes/s, FLOP/s and cost per second).

The attention stage built in this repository is the operator whose time the model takes to be
"memory traffic divided by memory bandwidth"; `attention_latency` evaluates that roofline with
either a nominal beta or the effective bandwidth measured by `profile_table.py`.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Iterable, Sequence, Tuple


@dataclasses.dataclass(frozen=True)
class Gpu:
    name: str
    cost: float       # c: monetary cost per unit time
    beta: float       # memory bandwidth, bytes per unit time
    mem: float        # M: memory capacity, bytes
    flops: float      # F: peak compute, FLOP per unit time

    @property
    def alpha(self) -> float:
        """Cost per byte of memory traffic, c / beta (Section 3.1)."""
        return self.cost / self.beta

    @property
    def gamma(self) -> float:
        """Cost per FLOP, c / F (Section 3.1)."""
        return self.cost / self.flops


def gpu_from_table(name: str, bw_gbs: float, mem_gb: float, tflops: float, dollars_per_hour: float) -> Gpu:
    """A GPU type from the units Table 1 uses (GB/s, GB, BF16 TFLOPS, $/GPU-h); cost per second."""
    return Gpu(name, dollars_per_hour / 3600.0, bw_gbs * 1e9, mem_gb * 1e9, tflops * 1e12)


# ----------------------------------------------------------------- operator roofline ---

def operator_latency(bytes_loaded: float, flop: float, beta: float, flops: float) -> float:
    """Appendix A.1: T(o) = max(D / beta, W / F)."""
    return max(bytes_loaded / beta, flop / flops)


def attention_latency(batch: float, m_kv: float, beta: float) -> float:
    """Appendix A.4 with the memory-bound assumption of Appendix A.2: D_attn(b) ~ b * m_kv(s),
    latency = D_attn / beta."""
    return batch * m_kv / beta


def kv_bytes_per_request(seq_len: float, layers: int, num_kv_heads: int, head_dim: int, bytes_per_elem: int = 2,
                         window: int = 0) -> float:
    """m_kv(s) of a stack of identical attention layers: K and V rows of the visible keys
    (a sliding-window layer sees min(s, W) keys -- Section 3.4, "a bounded window")."""
    visible = min(seq_len, window) if window > 0 else seq_len
    return layers * 2.0 * num_kv_heads * head_dim * bytes_per_elem * visible


# ------------------------------------------------------------------ Eq. 1-4, threshold ---

def cpt_hom(gpu: Gpu, m_kv: float, p_act: float) -> float:
    """Eq. 1: homogeneous ODS on one GPU type: alpha * m_kv(s) + 2 * gamma * P_act."""
    return gpu.alpha * m_kv + 2.0 * gpu.gamma * p_act


def cpt_het(gpu_attn: Gpu, gpu_gemm: Gpu, m_kv: float, p_act: float) -> float:
    """Eq. 2: attention on type j, GEMM-dominated operators on type k."""
    return gpu_attn.alpha * m_kv + 2.0 * gpu_gemm.gamma * p_act


def batch_limit(gpu: Gpu, m_weights: float, m_kv: float) -> Tuple[float, int]:
    """Eq. 3: relaxed colocated batch limit b_bar = (M - M_weights) / m_kv and its floor b_max."""
    b_bar = (gpu.mem - m_weights) / m_kv
    return b_bar, int(math.floor(b_bar))


def cpt_coloc(gpu: Gpu, m_kv: float, p_act: float, m_weights: float) -> float:
    """Eq. 4: colocated serving at the largest relaxed batch:
    alpha * m_kv + max(alpha * M_weights / b_bar, 2 * gamma * P_act)."""
    b_bar, _ = batch_limit(gpu, m_weights, m_kv)
    if b_bar <= 0:
        return math.inf
    return gpu.alpha * m_kv + max(gpu.alpha * m_weights / b_bar, 2.0 * gpu.gamma * p_act)


def gemm_threshold(gpu: Gpu, m_weights: float, p_act: float) -> float:
    """b* = M_weights * F / (2 * P_act * beta): the batch at which GEMM turns compute-bound."""
    return m_weights * gpu.flops / (2.0 * p_act * gpu.beta)


# ------------------------------------------------------------------------- Theorem 1 ---

def gain_hom(gpu: Gpu, m_kv: float, p_act: float, m_weights: float) -> float:
    """G_hom(s) = CPT_coloc(s) / CPT_hom(s) (Section 3.2)."""
    return cpt_coloc(gpu, m_kv, p_act, m_weights) / cpt_hom(gpu, m_kv, p_act)


def gain_hom_bound(gpu: Gpu, m_weights: float) -> float:
    """Theorem 1, part 3: G_hom(s) < M / (M - M_weights)."""
    return gpu.mem / (gpu.mem - m_weights)


# ------------------------------------------------------------------------- Theorem 2 ---

def cpt_hom_star(gpus: Iterable[Gpu], m_kv: float, p_act: float) -> float:
    """Eq. 5: the best single type."""
    return min(cpt_hom(g, m_kv, p_act) for g in gpus)


def cpt_het_star(gpus: Sequence[Gpu], m_kv: float, p_act: float) -> float:
    """Eq. 6: attention on the type with the lowest cost per byte, GEMMs on the type with the
    lowest cost per FLOP."""
    return min(g.alpha for g in gpus) * m_kv + min(g.gamma for g in gpus) * 2.0 * p_act


def gain_het(gpus: Sequence[Gpu], m_kv: float, p_act: float) -> float:
    """G_het(s) = CPT_hom_star / CPT_het_star (Section 3.3)."""
    return cpt_hom_star(gpus, m_kv, p_act) / cpt_het_star(gpus, m_kv, p_act)


def hardware_ratio(a: Gpu, b: Gpu) -> float:
    """eta = (beta_1 F_2) / (beta_2 F_1), labelled so that eta >= 1 (Section 3.3)."""
    eta = (a.beta * b.flops) / (b.beta * a.flops)
    return eta if eta >= 1.0 else 1.0 / eta


def gain_het_bound(a: Gpu, b: Gpu) -> float:
    """Theorem 2, part 3: G_het(s) <= (1 + sqrt(eta)) / 2."""
    return (1.0 + math.sqrt(hardware_ratio(a, b))) / 2.0


def het_crossing(a: Gpu, b: Gpu, p_act: float) -> float:
    """Theorem 2, part 3: x* = 2 P_act (gamma_1 - gamma_2) / (alpha_2 - alpha_1), the value of
    m_kv at which the two homogeneous costs cross (type 1 is the one with the smaller alpha).
    Returns inf when one type dominates the other on both metrics."""
    g1, g2 = (a, b) if a.alpha <= b.alpha else (b, a)
    if g1.gamma <= g2.gamma:
        return math.inf
    return 2.0 * p_act * (g1.gamma - g2.gamma) / (g2.alpha - g1.alpha)


# --------------------------------------------------------------- CAD feasibility (App. A.6) ---

def cad_attn_latency_max(gpu_attn: Gpu, microbatches: int) -> float:
    """T_attn_max = M_1 / (mu * beta_1): each of mu microbatches can hold at most M_1 / mu bytes."""
    return gpu_attn.mem / (microbatches * gpu_attn.beta)


def cad_rest_latency_min(gpu_rest: Gpu, m_weights_per_gpu: float) -> float:
    """T_rest_min = M_weights,2 / beta_2: the rest-of-model stage must at least load its weights."""
    return m_weights_per_gpu / gpu_rest.beta


def cad_feasible(gpu_attn: Gpu, microbatches: int, gpu_rest: Gpu, m_weights_per_gpu: float) -> bool:
    """Necessary condition for balanced CAD: M_1 / (mu beta_1) >= M_weights,2 / beta_2."""
    return cad_attn_latency_max(gpu_attn, microbatches) >= cad_rest_latency_min(gpu_rest, m_weights_per_gpu)


def with_measured_bandwidth(gpu: Gpu, beta_eff: float) -> Gpu:
    """The same GPU type with the bandwidth the attention stage actually sustains."""
    return dataclasses.replace(gpu, beta=beta_eff)


# ------------------------------------------------ measured profile -> latency model ---

def fit_affine_latency(points: Sequence[Tuple[float, float]], relative: bool = True) -> Tuple[float, float]:
    """Least-squares fit of T = t0 + D / beta to measured (bytes D, latency T) pairs of an attention stage.

    The paper's roofline for the operator is T = D / beta (Appendix A.1, A.4); a measured stage also has a
    latency floor t0 (first-tile latency, tail, combine) that matters for the small steps a stage runs when
    it holds few microbatches under a tight time-per-output-token target (Section 4: stage latencies come
    from profiled execution latency).  `relative` weights every point by 1 / T^2, i.e. minimises the relative
    error, so that microsecond-sized steps count as much as millisecond-sized ones.  Returns (t0, beta) in the
    units of the inputs."""
    pts = [(float(d), float(t)) for d, t in points]
    if len(pts) < 2:
        raise ValueError("need at least two measured points")
    if any(t <= 0.0 for _, t in pts):
        raise ValueError("latencies must be positive")
    w = [1.0 / (t * t) if relative else 1.0 for _, t in pts]
    sw = sum(w)
    sx = sum(wi * d for wi, (d, _) in zip(w, pts))
    sy = sum(wi * t for wi, (_, t) in zip(w, pts))
    sxx = sum(wi * d * d for wi, (d, _) in zip(w, pts))
    sxy = sum(wi * d * t for wi, (d, t) in zip(w, pts))
    den = sw * sxx - sx * sx
    if den <= 1e-12 * sw * sxx:
        raise ValueError("the points need at least two distinct sizes")
    slope = (sw * sxy - sx * sy) / den
    if slope <= 0.0:
        raise ValueError("latency does not grow with the bytes loaded")
    return (sy - slope * sx) / sw, 1.0 / slope


def attention_latency_affine(batch: float, m_kv: float, t0: float, beta: float) -> float:
    """The profiled form of `attention_latency`: a latency floor plus memory traffic over bandwidth."""
    return t0 + batch * m_kv / beta
