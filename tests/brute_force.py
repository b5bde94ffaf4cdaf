"""Dense float64 numpy evaluation of the method, written straight from Eq. 1-3 of the paper.

Independent of the C oracle (shares no code with it): an explicit DCT-II matrix, explicit 0/1 masks, full
reconstructed key matrices and the literal logit difference of Eq. 2.  Only usable on small inputs.
"""
from __future__ import annotations

import numpy as np


def dct_matrix(B: int) -> np.ndarray:
    """Orthonormal DCT-II basis F_B (rows = frequencies)."""
    F = np.zeros((B, B))
    for k in range(B):
        s = np.sqrt(1.0 / B) if k == 0 else np.sqrt(2.0 / B)
        for n in range(B):
            F[k, n] = s * np.cos(np.pi * (2 * n + 1) * k / (2 * B))
    return F


def stored_coefficients(x0, x1, bf16: bool):
    """Coefficients as the cache stores them: float32 add/sub, one float32 multiply, storage rounding."""
    c32 = np.float32(np.sqrt(0.5))
    z0 = (x0.astype(np.float32) + x1.astype(np.float32)) * c32
    z1 = (x0.astype(np.float32) - x1.astype(np.float32)) * c32
    if bf16:
        z0, z1 = _rne_bf16(z0), _rne_bf16(z1)
    return z0.astype(np.float32), z1.astype(np.float32)


def _rne_bf16(x):
    import torch  # library rounding, independent of both implementations

    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def kept_mask(z1, k: int) -> np.ndarray:
    """0/1 mask of the k largest |z1| entries, ties to the lowest flat index (stable argsort)."""
    mag = np.abs(z1.astype(np.float64)).ravel()
    order = np.argsort(-mag, kind="stable")
    m = np.zeros(mag.size)
    m[order[:k]] = 1.0
    return m.reshape(z1.shape)


def candidates(z0, z1, mask, x_pair):
    """Eq. 3: X~ = F^T [Z0 ; 1_S Z1] for S = empty (shared), the kept set (residual); exact = original."""
    F = dct_matrix(2)
    Z_sh = np.stack([z0.astype(np.float64), np.zeros_like(z0, dtype=np.float64)])
    Z_rs = np.stack([z0.astype(np.float64), mask * z1.astype(np.float64)])
    X_sh = np.einsum("kl,ktc->ltc", F, Z_sh)  # F^T Z
    X_rs = np.einsum("kl,ktc->ltc", F, Z_rs)
    X_ex = np.stack([x_pair[0].astype(np.float64), x_pair[1].astype(np.float64)])
    return X_sh, X_rs, X_ex


def probe_errors(z0k, z1k, mask, q_pair, group: int, h: int, pos):
    """Eq. 2 error term, literal: mean over (layer, group head, probe query) of ||Q Khat^T - Q K^T||^2 / d,
    keys restricted to j <= pos (causal), with K = F^T Z of the stored coefficients."""
    F = dct_matrix(2)
    d = z0k.shape[1]
    K = np.einsum("kl,ktc->ltc", F, np.stack([z0k, z1k]).astype(np.float64))
    X_sh, X_rs, _ = candidates(z0k, z1k, mask, (z0k, z0k))
    T = z0k.shape[0]
    causal = (np.arange(T)[None, :] <= np.asarray(pos)[:, None]).astype(np.float64)  # [W, T]
    out = []
    for Khat in (X_sh, X_rs):
        tot, cnt = 0.0, 0
        for layer in range(2):
            for g in range(group):
                Q = q_pair[layer][:, h * group + g, :].astype(np.float64)  # [W, d]
                diff = (Q @ Khat[layer].T) / np.sqrt(d) - (Q @ K[layer].T) / np.sqrt(d)
                tot += float(np.sum((diff * causal) ** 2))
                cnt += Q.shape[0]
        out.append(tot / cnt)
    return out[0], out[1]


def attention(khat, vhat, q):
    d = khat.shape[1]
    logit = khat @ q.astype(np.float64) / np.sqrt(d)
    p = np.exp(logit - logit.max())
    return (p @ vhat) / p.sum()


def token_scores(z0k, z1k, q_pair, group: int, h: int, pos):
    """The unnumbered token score between Eq. 2 and Eq. 3, literally: s_t = max over the probe queries that can see t
    (and over the block's layers and the group's heads) of |Q (K_t - Khat_t^shared)^T|, with K = F^T [Z0; Z1] the key
    rows the stored coefficients stand for and Khat^shared = F^T [Z0; 0] the shared-depth candidate of Eq. 3 (S empty).
    No 1/sqrt(d): the printed score has none."""
    F = dct_matrix(2)
    Z = np.stack([z0k, z1k]).astype(np.float64)
    Z_shared = np.stack([z0k.astype(np.float64), np.zeros_like(z1k, dtype=np.float64)])
    K = np.einsum("kl,ktc->ltc", F, Z)                # F^T Z: [layer, T, d]
    K_shared = np.einsum("kl,ktc->ltc", F, Z_shared)
    T = z1k.shape[0]
    best = np.zeros(T)
    visible = np.arange(T)[None, :] <= np.asarray(pos)[:, None]  # [W, T]
    for layer in range(2):
        for g in range(group):
            Q = q_pair[layer][:, h * group + g, :].astype(np.float64)
            s = np.abs(Q @ (K[layer] - K_shared[layer]).T)      # [W, T]
            s = np.where(visible, s, 0.0)
            best = np.maximum(best, s.max(axis=0))
    return best
