"""Vocabulary-sharded form of the verification step in plain numpy fp64 (TEST INFRASTRUCTURE).

Each shard holds a contiguous range of columns of every row.  The three local phases follow the
step of Sec. 3.2 / 3.1 with every quantity that needs the whole row rebuilt from per-shard pieces:
  stats   per row: m = max of the local logits, s = sum exp((l - m)/T), the draft token's logit
          if its column is local;
  decide  M = max_r m_r, Z = sum_r s_r exp((m_r - M)/T); P(x) = exp((l_x - M)/T) / Z;
          max P_t = 1/Z_t; the rule of Sec. 3.2 with the uniforms of the unsharded oracle; then
          the local mass of the row to draw from (residual max(0, P_t - P_d) after a rejection,
          P_t of row K otherwise);
  pick    the shard whose columns contain the point u S of the cumulative mass (shards in
          vocabulary order) walks its own columns to the token.
It must reproduce the unsharded oracle (``ears_oracle.c``) for any split; that invariance is its pin.
The uniforms come from the C oracle's counter-based generator.
"""
from __future__ import annotations

import numpy as np

from . import ears_oracle as _o

EPS = 1e-10


def _np(a):
    if isinstance(a, np.ndarray):
        return a
    import torch
    if a.dtype in (torch.bfloat16, torch.float16):
        a = a.float()
    return a.detach().cpu().numpy()


class OracleShardStep:
    def __init__(self, target_shard, draft_shard, draft_tokens, v_first, V, temperature, beta,
                 seed=0, offset=0, b_first=0):
        self.t = _np(target_shard).astype(np.float64)
        self.d = _np(draft_shard).astype(np.float64)
        self.x = _np(draft_tokens).astype(np.int64)
        self.B, K1, self.Vs = self.t.shape
        self.K = K1 - 1
        self.v_first, self.V = int(v_first), int(V)
        self.T, self.beta = float(temperature), float(beta)
        self.seed, self.offset, self.b_first = int(seed), int(offset), int(b_first)

    def _row(self, b, r):
        return self.t[b, r] if r <= self.K else self.d[b, r - self.K - 1]

    def stats(self):
        """-> [B (2K+1), 4] float64 (m, s, token logit, 1 if the token's column is local)."""
        B, K, R = self.B, self.K, 2 * self.K + 1
        out = np.zeros((B * R, 4))
        for b in range(B):
            for r in range(R):
                row = self._row(b, r)
                m = np.max(row)                      # NaN if the row holds one
                s = 0.0
                if np.isfinite(m):
                    for l in row:                    # summed left to right
                        s += np.exp((l - m) / self.T)
                elif np.isnan(m) or m == np.inf:
                    s = np.nan
                o = out[b * R + r]
                o[0], o[1] = m, s
                if r != K:
                    tok = self.x[b, r if r < K else r - K - 1] - self.v_first
                    if 0 <= tok < self.Vs:
                        o[2], o[3] = row[tok], 1.0
        return _as_torch(out)

    def _combine(self, all_stats, b, r):
        q = all_stats[:, b * (2 * self.K + 1) + r, :]
        M = np.max(q[:, 0])
        if not np.isfinite(M):
            return M, np.nan, 0.0, 0
        Z = 0.0
        for m, s in q[:, :2]:
            if m > -np.inf:
                Z += s * np.exp((m - M) / self.T)
        owners = int(np.sum(q[:, 3] != 0))
        l = float(q[q[:, 3] != 0, 2][0]) if owners else 0.0
        return M, Z, l, owners

    def decide(self, all_stats):
        """all_stats [n_shards, B (2K+1), 4] -> [B] local mass of the row each sequence draws from."""
        A = _np(all_stats).astype(np.float64)
        B, K = self.B, self.K
        self.acc = np.full(B, -1, np.int32)
        self.tok = np.full((B, K + 1), -1, np.int32)
        self.norm = [None] * B
        mass = np.zeros(B)
        for b in range(B):
            rows = [self._combine(A, b, r) for r in range(2 * K + 1)]
            valid = all(np.isfinite(M) and Z > 0 and np.isfinite(Z) for M, Z, _, _ in rows)
            n = K
            for k in range(K):
                if not valid:
                    break
                Mt, Zt, lt, ot = rows[k]
                Md, Zd, ld, od = rows[K + 1 + k]
                if not (0 <= self.x[b, k] < self.V) or ot != 1 or od != 1:
                    valid = False
                    break
                pt = np.exp((lt - Mt) / self.T) / Zt
                pd = np.exp((ld - Md) / self.T) / Zd
                R = pt / max(pd, EPS)                       # Sec. 3.2 step 2, Sec. 3.3 item 2
                tol = self.beta * (1.0 - 1.0 / Zt)          # max P_t = exp(0) / Z_t
                U = _o.uniform_accept(self.seed, self.offset, self.b_first + b, k)
                if not R >= max(U - tol, 0.0) and n == K:
                    n = k
            if not valid:
                continue
            self.acc[b] = n
            self.tok[b, :n] = self.x[b, :n]
            Mt, Zt, _, _ = rows[n]
            pt = np.exp((self.t[b, n] - Mt) / self.T) / Zt
            if n < K:
                Md, Zd, _, _ = rows[K + 1 + n]
                pd = np.exp((self.d[b, n] - Md) / self.T) / Zd
                local = np.where(pt > pd, pt - pd, 0.0)
            else:
                local = pt
            self.norm[b] = (local, pt)
            mass[b] = np.cumsum(local)[-1]
        return _as_torch(mass)

    def pick(self, rank, all_stats, all_mass):
        """-> (accept_len, tokens); tokens[b, n] is set only on the shard that owns the draw."""
        A = _np(all_stats).astype(np.float64)
        Mss = _np(all_mass).astype(np.float64)
        K = self.K
        for b in range(self.B):
            n = self.acc[b]
            if n < 0:
                continue
            masses = Mss[:, b].copy()
            local, pt = self.norm[b]
            if n < K and np.sum(masses) < 1e-300:     # defensive, as in the unsharded oracle: use P_t
                M, Z, _, _ = self._combine(A, b, n)
                q = A[:, b * (2 * K + 1) + n, :]
                masses = np.array([s * np.exp((m - M) / self.T) / Z if m > -np.inf else 0.0 for m, s in q[:, :2]])
                local = pt
            u = _o.uniform_final(self.seed, self.offset, self.b_first + b, K)
            target = u * np.cumsum(masses)[-1]
            cum, owner, before, lastpos, before_last = 0.0, -1, 0.0, -1, 0.0
            for r, v in enumerate(masses):
                if v > 0:
                    lastpos, before_last = r, cum
                if owner < 0 and v > 0 and target < cum + v:
                    owner, before = r, cum
                cum += v
            if owner < 0:
                owner, before = lastpos, before_last
            if owner != rank:
                continue
            c = np.cumsum(local)
            hit = np.nonzero((target - before < c) & (local > 0))[0]
            j = hit[0] if hit.size else np.nonzero(local > 0)[0][-1]
            self.tok[b, n] = self.v_first + j
        return _as_torch(self.acc), _as_torch(self.tok)


def _as_torch(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a))
