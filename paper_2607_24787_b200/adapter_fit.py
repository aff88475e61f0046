"""Closed-form stand-ins for trained adapter weights (data preparation only: the adapters they
produce run through the same kernels as any other A / B_up pair).

The paper trains each layer's adapter to match the next layer's router distribution (Section 3.4).
Without its corpus and models, three substitutes of the same shape are offered:

* gate reuse   A = W_r^{l+1}, B_up = I (rank n): the training-free predictor the paper compares with;
* truncated SVD of W_r^{l+1} at the adapter's rank: the best rank-r approximation of that gate in
  the Frobenius norm, which ignores the data distribution;
* reduced-rank ridge regression of the next layer's router logits on this layer's router input over
  a calibration stream: the rank-r linear map with the smallest squared logit error on that stream
  (the classical closed form: ridge fit, then projection of the fitted values onto their leading
  right singular vectors).
"""
from __future__ import annotations

import torch


def svd_adapter(w_next: torch.Tensor, rank: int):
    """Rank-`rank` factors of the next layer's gate matrix w_next [n, D].

    Returns (A [rank, D], B_up [n, rank]) in fp32 with B_up @ A the truncated SVD of w_next; the
    singular values are split evenly between the two factors so both stay in a narrow range."""
    u, s, vh = torch.linalg.svd(w_next.double(), full_matrices=False)
    r = min(rank, s.numel())
    root = s[:r].sqrt()
    a = (root[:, None] * vh[:r]).float()
    b = (u[:, :r] * root[None, :]).float()
    if r < rank:      # pad with zero directions so the shapes match the requested rank
        a = torch.cat((a, a.new_zeros(rank - r, a.shape[1])))
        b = torch.cat((b, b.new_zeros(b.shape[0], rank - r)), dim=1)
    return a.contiguous(), b.contiguous()


def reduced_rank_fit(x: torch.Tensor, z: torch.Tensor, rank: int, ridge: float = 1e-3):
    """Rank-`rank` map from x [N, D] to z [N, n] minimising ||z - x C||_F^2 + ridge' ||C||_F^2.

    `ridge` is relative to the mean squared row norm of x. Returns (A [rank, D], B_up [n, rank]),
    fp32, with C = A^T B_up^T. The ridge solution is formed in its dual (N x N) form, so N may be
    far smaller than D."""
    xd, zd = x.double(), z.double()
    n_rows = xd.shape[0]
    gram = xd @ xd.T
    lam = ridge * gram.diagonal().mean()
    alpha = torch.linalg.solve(gram + lam * torch.eye(n_rows, dtype=gram.dtype, device=gram.device), zd)
    c_full = xd.T @ alpha                                  # [D, n] ridge solution
    fitted = xd @ c_full                                   # [N, n]
    _, _, vh = torch.linalg.svd(fitted, full_matrices=False)
    r = min(rank, vh.shape[0])
    v = vh[:r].T                                           # [n, r] leading right singular vectors
    a = (c_full @ v).T                                     # [r, D]
    b = v                                                  # [n, r]
    # balance the two factors (bf16 storage): scale each direction so |A_i| = |B_i|
    na = a.norm(dim=1).clamp_min(1e-30)
    nb_ = b.norm(dim=0).clamp_min(1e-30)
    g = (nb_ / na).sqrt()
    a = a * g[:, None]
    b = b / g[None, :]
    if r < rank:
        a = torch.cat((a, a.new_zeros(rank - r, a.shape[1])))
        b = torch.cat((b, b.new_zeros(b.shape[0], rank - r)), dim=1)
    return a.float().contiguous(), b.float().contiguous()
