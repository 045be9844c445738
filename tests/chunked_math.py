"""fp64 numpy statement of the chunked (block-decomposed) form of the SSD layer, used only as a
test of the algebra the CUDA kernels rely on: it must agree with the per-timestep oracle to
rounding.  It is neither the oracle nor product code and shares nothing with either.

Per (b, h) and chunk of Q steps: a_t = dt_t*A, cs_t = inclusive cumsum of a inside the chunk,
H_in = state entering the chunk, Gout = dLoss/d(state leaving the chunk).
"""
import numpy as np


def chunked_fwd(x, dt, A, Bm, Cm, D, h0, Q):
    B, L, H, P = x.shape
    G, N = Bm.shape[2:]
    y = np.empty_like(x)
    hf = np.zeros((B, H, P, N))
    for b in range(B):
        for h in range(H):
            g = h // (H // G)
            Hin = np.zeros((P, N)) if h0 is None else h0[b, h].copy()
            for c0 in range(0, L, Q):
                sl = slice(c0, c0 + Q)
                xc, dtc, Bc, Cc = x[b, sl, h], dt[b, sl, h], Bm[b, sl, g], Cm[b, sl, g]
                cs = np.cumsum(dtc * A[h])
                w = np.exp(cs[-1] - cs) * dtc
                S = (xc * w[:, None]).T @ Bc
                diff = cs[:, None] - cs[None, :]
                Lm = np.where(np.tril(np.ones((Q, Q), bool)), np.exp(np.minimum(diff, 0.0)), 0.0)
                M = (Cc @ Bc.T) * Lm * dtc[None, :]
                y[b, sl, h] = M @ xc + np.exp(cs)[:, None] * (Cc @ Hin.T) + D[h] * xc
                Hin = np.exp(cs[-1]) * Hin + S
            hf[b, h] = Hin
    return y, hf


def chunked_bwd(x, dt, A, Bm, Cm, D, h0, dy, dh_final, Q):
    B, L, H, P = x.shape
    G, N = Bm.shape[2:]
    nc = L // Q
    dx = np.empty_like(x)
    ddt = np.empty_like(dt)
    dB = np.zeros_like(Bm)
    dC = np.zeros_like(Cm)
    dA = np.zeros(H)
    dD = np.zeros(H)
    dh0 = np.zeros((B, H, P, N))
    for b in range(B):
        for h in range(H):
            g = h // (H // G)
            # recompute the chunk-entry states
            Hs = np.empty((nc + 1, P, N))
            Hs[0] = 0.0 if h0 is None else h0[b, h]
            css = []
            for c in range(nc):
                sl = slice(c * Q, (c + 1) * Q)
                cs = np.cumsum(dt[b, sl, h] * A[h])
                css.append(cs)
                w = np.exp(cs[-1] - cs) * dt[b, sl, h]
                Hs[c + 1] = np.exp(cs[-1]) * Hs[c] + (x[b, sl, h] * w[:, None]).T @ Bm[b, sl, g]
            carry = np.zeros((P, N)) if dh_final is None else dh_final[b, h].copy()
            for c in range(nc - 1, -1, -1):
                sl = slice(c * Q, (c + 1) * Q)
                xc, dtc, Bc, Cc, dyc = x[b, sl, h], dt[b, sl, h], Bm[b, sl, g], Cm[b, sl, g], dy[b, sl, h]
                cs = css[c]
                Gout = carry
                E = (dyc * np.exp(cs)[:, None]).T @ Cc
                carry = np.exp(cs[-1]) * Gout + E
                diff = cs[:, None] - cs[None, :]
                Lm = np.where(np.tril(np.ones((Q, Q), bool)), np.exp(np.minimum(diff, 0.0)), 0.0)  # [t, s]
                CB = Cc @ Bc.T
                wl = np.exp(cs[-1] - cs)
                u = (CB * Lm).T @ dyc + wl[:, None] * (Bc @ Gout.T)
                dx[b, sl, h] = D[h] * dyc + dtc[:, None] * u
                ddt_direct = np.sum(xc * u, axis=1)
                W = (dyc @ xc.T) * Lm * dtc[None, :]
                dB_intra, dB_inter = W.T @ Cc, (dtc * wl)[:, None] * (xc @ Gout)
                dCh = W @ Bc + np.exp(cs)[:, None] * (dyc @ Hs[c])
                dB[b, sl, g] += dB_intra + dB_inter
                dC[b, sl, g] += dCh
                # da_t = exp(a_t) <g_t, h_{t-1}> split by intra-/inter-chunk parts of g_t and h_{t-1}:
                # suffix sum of (rho - psi) [pairs t' >= t > s, and outputs reading the entry state],
                # exclusive prefix sum of psi2 [inputs before t feeding Gout], plus e^{cs_last}<Gout,H_in>
                rho = np.sum(Cc * dCh, axis=1)
                psi = np.sum(Bc * dB_intra, axis=1)
                psi2 = np.sum(Bc * dB_inter, axis=1)
                da = (np.cumsum((rho - psi)[::-1])[::-1] + (np.cumsum(psi2) - psi2)
                      + np.exp(cs[-1]) * np.sum(Gout * Hs[c]))
                ddt[b, sl, h] = ddt_direct + A[h] * da
                dA[h] += np.sum(dtc * da)
                dD[h] += np.sum(dyc * xc)
            dh0[b, h] = carry
    return dict(dx=dx, ddt=ddt, dA=dA, dB=dB, dC=dC, dD=dD, dh0=dh0)
