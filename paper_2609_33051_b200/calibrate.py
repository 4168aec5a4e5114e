"""Offline calibration of the sketching matrix and the fixed coefficient map (not on the hot path).

Given calibration effective queries q~_i of one head and the average state metric E_0 (Section 4.1):
z_i = E_0^{1/2} q~_i, C_z = mean z z^T, P_G = eigenvectors of the G largest eigenvalues (uncentered PCA),
Omega = E_0^{-1/2} P_G (Eq. 8 and Appendix A.1) and C_offline = (Omega^T E_0 Omega)^+ Omega^T E_0 (Eq. 10).
Runs once per head in float64 on the host with torch.linalg; its results are inputs of the CUDA library.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch


def _sym_sqrt_pair(E0: torch.Tensor, rcond: float = 1e-12) -> Tuple[torch.Tensor, torch.Tensor]:
    lam, P = torch.linalg.eigh(E0)
    keep = lam > rcond * lam.max()
    root = torch.where(keep, lam.clamp_min(0).sqrt(), torch.zeros_like(lam))
    iroot = torch.where(keep, 1.0 / root.clamp_min(1e-300), torch.zeros_like(lam))
    return (P * root) @ P.T, (P * iroot) @ P.T


def fit_head(queries: torch.Tensor, rank: int, E0: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Omega [K, rank] and C [rank, K] (float64) for one head from its calibration queries [N, K]."""
    Q = queries.to(torch.float64)
    K = Q.shape[1]
    E0 = torch.eye(K, dtype=torch.float64) if E0 is None else E0.to(torch.float64)
    E_half, E_ihalf = _sym_sqrt_pair(E0)
    Z = Q @ E_half
    lam, P = torch.linalg.eigh(Z.T @ Z / Z.shape[0])
    P = P.flip(1)[:, :rank]                                   # eigh is ascending
    idx = P.abs().argmax(dim=0)
    sign = torch.sign(P[idx, torch.arange(rank)])
    P = P * torch.where(sign == 0, torch.ones_like(sign), sign)
    Omega = E_ihalf @ P
    C = torch.linalg.pinv(Omega.T @ E0 @ Omega) @ Omega.T @ E0
    return Omega, C
