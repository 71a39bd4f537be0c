"""A second, independently written formulation of Algorithm 1 (numpy, fp64).

One pool of B_p + B_c token slots with no physical split between proximity and
context: a token is "in proximity" iff its position is among the B_p highest.
The new token takes the evicted token's slot.  The tests demand that this form
and the oracle's three-list form agree on every victim, every merge target and
every output -- which is what lets a device layout use a single slot pool.
"""
import numpy as np


class PoolCache:
    def __init__(self, d, G, Bp, Bc, Br, lam=0.98, alpha=1.0, scale=None):
        self.d, self.G, self.Bp, self.Bc, self.Br = d, G, Bp, Bc, Br
        self.lam, self.alpha = lam, alpha
        self.scale = scale if scale else 1.0 / np.sqrt(d)
        n = Bp + Bc
        self.K = np.zeros((n, d))
        self.V = np.zeros((n, d))
        self.s = np.zeros(n, dtype=np.float32)
        self.pos = np.full(n, -1, dtype=np.int64)
        self.n_live = 0
        self.Kr = np.zeros((Br, d))
        self.Vr = np.zeros((Br, d))
        self.w = np.zeros(Br, dtype=np.int64)
        self.n_res = 0
        self.T = 0

    def permute(self, rng):
        """Shuffle the physical slots; nothing observable may change."""
        p = rng.permutation(self.n_live)
        for a in (self.K, self.V, self.s, self.pos):
            a[: self.n_live] = a[: self.n_live][p]

    def step(self, q, k_new, v_new):
        n, r = self.n_live, self.n_res
        keys = np.concatenate([self.K[:n], self.Kr[:r], k_new[None]], axis=0)
        vals = np.concatenate([self.V[:n], self.Vr[:r], v_new[None]], axis=0)
        comp = np.zeros(n + r + 1)
        comp[n:n + r] = self.alpha * np.log(self.w[:r].astype(np.float64))
        logits = (q @ keys.T) * self.scale + comp[None, :]
        logits -= logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        a = p / p.sum(axis=1, keepdims=True)
        out = a @ vals
        mean_a = a.sum(axis=0) / self.G
        self.s[:n] = (self.lam * self.s[:n].astype(np.float64) + mean_a[:n]).astype(np.float32)
        s_new = np.float32(mean_a[-1])
        pos_new = self.T
        self.T += 1
        victim_pos, merge_slot = -1, -1
        if n + 1 <= self.Bp + self.Bc:
            self._put(n, k_new, v_new, s_new, pos_new)
            self.n_live += 1
            return out, victim_pos, merge_slot
        # candidates: everything no longer among the B_p latest positions
        cand = [(self.s[j], self.pos[j], j) for j in range(n) if self.pos[j] <= pos_new - self.Bp]
        if self.Bp == 0:
            cand.append((s_new, pos_new, -1))
        sv, pv, jv = min(cand, key=lambda c: (c[0], c[1]))
        victim_pos = int(pv)
        kc, vc = (k_new, v_new) if jv < 0 else (self.K[jv].copy(), self.V[jv].copy())
        if self.Br > 0:
            if self.n_res < self.Br:
                self.Kr[self.n_res], self.Vr[self.n_res], self.w[self.n_res] = kc, vc, 1
                self.n_res += 1
                merge_slot = -2
            else:
                dots = (self.Kr @ kc).astype(np.float32)
                merge_slot = int(np.argmax(dots))          # first maximum = lowest slot
                wr = float(self.w[merge_slot])
                self.Kr[merge_slot] = (wr * self.Kr[merge_slot] + kc) / (wr + 1.0)
                self.Vr[merge_slot] = (wr * self.Vr[merge_slot] + vc) / (wr + 1.0)
                self.w[merge_slot] += 1
        if jv >= 0:
            self._put(jv, k_new, v_new, s_new, pos_new)
        return out, victim_pos, merge_slot

    def _put(self, j, k, v, s, pos):
        self.K[j], self.V[j], self.s[j], self.pos[j] = k, v, s, pos
