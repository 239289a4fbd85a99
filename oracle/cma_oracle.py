"""CPU oracle for the search-distribution update of ESSA's loop.  TEST INFRASTRUCTURE ONLY.

Section 3, "Evolutionary optimization", says that after every candidate's reward is known CMA-ES "updates
(m, sigma, C) based on the reward rankings"; Algorithm 1 (the line after the <seed, reward> exchange) has every
worker perform that one update on identical state.  The paper prints no formulas for it (it cites Hansen's
CMA-ES and used a library), so this file states the textbook (mu/mu_w, lambda)-CMA-ES of Hansen's tutorial
("The CMA Evolution Strategy: A Tutorial", 2016), in fp64, step by step in the tutorial's order and notation
(n = dimension, lambda = population size, y_k = (x_k - m)/sigma):

  selection and recombination   weights w_i from ln((lambda+1)/2) - ln(i), i = 1..mu = floor(lambda/2), normalised
                                to sum 1 (non-negative weights only);  mu_eff = 1 / sum w_i^2;
                                <y>_w = sum_i w_i y_{i:lambda};  m <- m + c_m sigma <y>_w,  c_m = 1;
  step-size control             p_sigma <- (1-c_sigma) p_sigma + sqrt(c_sigma (2-c_sigma) mu_eff) C^{-1/2} <y>_w,
                                C^{-1/2} = B D^{-1} B^T;  sigma <- sigma exp((c_sigma/d_sigma)(|p_sigma|/E|N(0,I)| - 1));
  covariance matrix adaptation  h_sigma = [ |p_sigma| / sqrt(1-(1-c_sigma)^{2(g+1)}) < (1.4 + 2/(n+1)) E|N(0,I)| ];
                                p_c <- (1-c_c) p_c + h_sigma sqrt(c_c (2-c_c) mu_eff) <y>_w;
                                C <- (1 - c_1 - c_mu + (1-h_sigma) c_1 c_c (2-c_c)) C + c_1 p_c p_c^T
                                     + c_mu sum_i w_i y_{i:lambda} y_{i:lambda}^T;
  decomposition                 C = B diag(D^2) B^T (symmetric eigendecomposition, a library routine here),
                                eigenvalues ascending; the next population is m + sigma B (D .* z).

Readings taken where neither the paper nor the tutorial fixes a choice (listed in the design notes too):
rewards are MAXIMISED (the best candidate is the one with the largest reward); ties keep population order (the
candidate with the lower index ranks first); a NaN reward ranks below every number; non-negative recombination
weights (the tutorial's optional negative weights are not used); the decomposition is refreshed on every update;
y_k is taken from the population as stored (fp32 table) and the state's own m and sigma; the default strategy
parameters are the tutorial's (alpha_cov = 2).

Pins (tests/test_cma_oracle_pins.py): closed forms of the weights and mu_eff; c_1 = c_mu = 0 leaves C unchanged;
invariance under strictly increasing transforms of the rewards; symmetric positive-definite C and B D^2 B^T = C;
the equal-weights, p_c = 0 special case where the rank-mu term is a sample covariance (numpy.cov); with sigma-path
learning rate zero the step size is unchanged; C^{-1/2} <y>_w equals B sum w_i z_i for a population drawn as
m + sigma B (D .* z); convergence on the sphere function to 1e-10 within a bounded number of generations.
Parity unpinned: the paper prints no worked numeric example of an update.

Only tests may import this module.  It shares no code with the CUDA library and imports nothing from it.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np


@dataclass
class CmaParams:
    """Strategy parameters of the tutorial's default setting for dimension n and population size lam."""

    n: int
    lam: int
    mu: int
    weights: np.ndarray  # [mu], positive, sum 1, decreasing
    mu_eff: float
    c_sigma: float
    d_sigma: float
    c_c: float
    c_1: float
    c_mu: float
    c_m: float
    chi_n: float  # E|N(0, I_n)|, the tutorial's approximation


def default_params(n: int, lam: int) -> CmaParams:
    """Tutorial, "default strategy parameters": selection/recombination, step-size control, covariance adaptation."""
    if n < 1 or lam < 2:
        raise ValueError("need n >= 1 and lambda >= 2")
    mu = lam // 2
    i = np.arange(1, mu + 1, dtype=np.float64)
    w_prime = np.log((lam + 1) / 2.0) - np.log(i)
    weights = w_prime / np.sum(w_prime)
    mu_eff = 1.0 / float(np.sum(weights * weights))
    c_sigma = (mu_eff + 2.0) / (n + mu_eff + 5.0)
    d_sigma = 1.0 + 2.0 * max(0.0, np.sqrt((mu_eff - 1.0) / (n + 1.0)) - 1.0) + c_sigma
    c_c = (4.0 + mu_eff / n) / (n + 4.0 + 2.0 * mu_eff / n)
    alpha_cov = 2.0
    c_1 = alpha_cov / ((n + 1.3) ** 2 + mu_eff)
    c_mu = min(1.0 - c_1, alpha_cov * (mu_eff - 2.0 + 1.0 / mu_eff) / ((n + 2.0) ** 2 + alpha_cov * mu_eff / 2.0))
    chi_n = np.sqrt(n) * (1.0 - 1.0 / (4.0 * n) + 1.0 / (21.0 * n * n))
    return CmaParams(n, lam, mu, weights, mu_eff, float(c_sigma), float(d_sigma), float(c_c), float(c_1), float(c_mu),
                     1.0, float(chi_n))


@dataclass
class CmaState:
    """(m, sigma, C) of Section 3 plus the evolution paths and the decomposition C = B diag(D^2) B^T."""

    mean: np.ndarray            # [n]
    sigma: float                # global step size
    C: np.ndarray               # [n, n] symmetric
    p_sigma: np.ndarray         # [n]
    p_c: np.ndarray             # [n]
    B: np.ndarray               # [n, n], columns = eigenvectors
    D: np.ndarray               # [n], square roots of the eigenvalues, ascending
    generation: int = 0
    params: Optional[CmaParams] = field(default=None, repr=False)


def decompose(C: np.ndarray):
    """C = B diag(D^2) B^T with eigenvalues ascending (library routine for symmetric matrices)."""
    lam, B = np.linalg.eigh(np.asarray(C, dtype=np.float64))
    return B, np.sqrt(np.maximum(lam, 0.0))


def init_state(mean0, sigma0: float, lam: int, C0=None, params: Optional[CmaParams] = None) -> CmaState:
    """Algorithm 1, "common CMA-ES state (m_0, sigma_0, C_0)": C_0 = I unless given, both paths zero."""
    mean0 = np.asarray(mean0, dtype=np.float64).copy()
    n = mean0.shape[0]
    C = np.eye(n) if C0 is None else np.asarray(C0, dtype=np.float64).copy()
    B, D = decompose(C)
    return CmaState(mean0, float(sigma0), C, np.zeros(n), np.zeros(n), B, D, 0, params or default_params(n, lam))


def rank_rewards(rewards) -> np.ndarray:
    """order[i] = index of the candidate with the (i+1)-th LARGEST reward; ties keep population order; NaN last."""
    r = np.asarray(rewards, dtype=np.float64)
    key = np.where(np.isnan(r), -np.inf, r)
    return np.argsort(-key, kind="stable")


def tell(state: CmaState, population, rewards) -> CmaState:
    """One update of (m, sigma, C) from a population x[lam, n] (as stored) and its rewards F[lam]; returns the new state."""
    p = state.params
    x = np.asarray(population, dtype=np.float64)
    n, lam = p.n, p.lam
    if x.shape != (lam, n):
        raise ValueError("population must be [lambda, n]")
    order = rank_rewards(rewards)
    y = (x[order[:p.mu]] - state.mean[None, :]) / state.sigma           # y_{i:lambda}, i = 1..mu
    y_w = p.weights @ y                                                 # <y>_w
    mean = state.mean + p.c_m * state.sigma * y_w
    # step-size control
    c_inv_sqrt_yw = state.B @ ((state.B.T @ y_w) / state.D)             # C^{-1/2} <y>_w = B D^{-1} B^T <y>_w
    p_sigma = (1.0 - p.c_sigma) * state.p_sigma + np.sqrt(p.c_sigma * (2.0 - p.c_sigma) * p.mu_eff) * c_inv_sqrt_yw
    norm_ps = float(np.sqrt(np.sum(p_sigma * p_sigma)))
    sigma = state.sigma * float(np.exp((p.c_sigma / p.d_sigma) * (norm_ps / p.chi_n - 1.0)))
    # covariance matrix adaptation
    g1 = state.generation + 1
    # (written without the division so that c_sigma = 0 is a legal setting)
    h_sigma = 1.0 if norm_ps < (1.4 + 2.0 / (n + 1.0)) * p.chi_n * np.sqrt(1.0 - (1.0 - p.c_sigma) ** (2 * g1)) else 0.0
    p_c = (1.0 - p.c_c) * state.p_c + h_sigma * np.sqrt(p.c_c * (2.0 - p.c_c) * p.mu_eff) * y_w
    delta_h = (1.0 - h_sigma) * p.c_c * (2.0 - p.c_c)
    rank_mu = np.zeros((n, n))
    for i in range(p.mu):
        rank_mu += p.weights[i] * np.outer(y[i], y[i])
    C = (1.0 - p.c_1 - p.c_mu + p.c_1 * delta_h) * state.C + p.c_1 * np.outer(p_c, p_c) + p.c_mu * rank_mu
    B, D = decompose(C)
    return CmaState(mean, sigma, C, p_sigma, p_c, B, D, g1, p)


def ask_from_normals(state: CmaState, z: np.ndarray) -> np.ndarray:
    """x_k = m + sigma B (D .* z_k) for given standard-normal rows z[lam, n] (Section 3: x ~ N(m, sigma^2 C))."""
    return state.mean[None, :] + state.sigma * (z * state.D[None, :]) @ state.B.T
