"""The FREE sampling loop (Algorithm 1) in fp64 (TEST INFRASTRUCTURE ONLY).

Conventions.  N transitions n = 1..N take x_0 ~ N(0, I) to x_N; transition n uses
schedule index s = N - n.  K drafts are proposed per round (Algorithm 1 drafts
t = a+1 .. b+1 with b = min(T, a+L): L+1 = K drafts; the packed target pass sees the
current state plus the first K-1 drafts and returns K means, as in Fig. 1).
Readings taken where the printed algorithm is inconsistent:
  * the cursor moves to one past the last finalised state (a <- j+1), so that the
    next target step consumes the verified / reflected state rather than
    recomputing it;
  * the last transition has sigma = 0 and is never drafted (b = min(N-1, a+K));
    the target takes it deterministically;
  * noise and uniforms are indexed by (transition, role), so a transition that is
    re-drafted after an earlier rejection reuses its draft-role noise.
"""
import numpy as np

from . import verify


def sample(x0, N, K, target_fn, draft_fn, sigma2, noise_target, noise_draft, uniforms,
           lam=None, trace=None, observe=None):
    """Run one trajectory.

    target_fn(x, s)              -> (mean, feature)          one target evaluation at schedule index s
    target_fn.packed(xs, ss)     -> means                     optional batched form (else called per state)
    draft_fn(x_prev, f_prev, s)  -> (mean_hat, feature_next)
    sigma2[s]; noise_target[n-1], noise_draft[n-1] of x0's shape; uniforms[n-1]; lam[n-1] or None.
    observe(t, m_hat_t, m_t, ell), if given, is called for every examined draft (used by the offline
    uncertainty run of Sec. 3.4).
    K == 0 is the plain sequential sampler.  Returns (x_N, stats).
    """
    x = np.asarray(x0, np.float64)
    stats = {"rounds": 0, "target_calls": 0, "draft_calls": 0, "accepted": 0, "rejected": 0,
             "accept_hist": np.zeros(max(K, 1) + 1, dtype=np.int64)}
    a = 1
    while a <= N:
        s_a = N - a
        m_a, f = target_fn(x, s_a)
        stats["target_calls"] += 1
        stats["rounds"] += 1
        x = m_a + np.sqrt(sigma2[s_a]) * np.asarray(noise_target[a - 1], np.float64)
        b = min(N - 1, a + K)
        if K == 0 or b <= a:
            a += 1
            continue
        # drafting: x_hat[t], t = a+1..b, from (x_hat[t-1], f[t-1])
        x_hat, m_hat = {a: x}, {}
        for t in range(a + 1, b + 1):
            s_t = N - t
            m_hat[t], f = draft_fn(x_hat[t - 1], f, s_t)
            stats["draft_calls"] += 1
            x_hat[t] = m_hat[t] + np.sqrt(sigma2[s_t]) * np.asarray(noise_draft[t - 1], np.float64)
        # one packed target pass over (x_hat[a], .., x_hat[b-1]) gives the target means m[a+1..b]
        ts = list(range(a + 1, b + 1))
        m = {t: target_fn(x_hat[t - 1], N - t)[0] for t in ts}
        stats["target_calls"] += 1
        # sequential verification, break at the first rejection
        j = a
        for t in ts:
            lam_t = 1.0 if lam is None else float(lam[t - 1])
            x, ok, ell = verify.verification(m_hat[t], m[t], sigma2[N - t], x_hat[t], uniforms[t - 1], lam_t)
            if trace is not None:
                trace.append((t, ok, ell))
            if observe is not None:
                observe(t, m_hat[t], m[t], ell)
            j = t
            if not ok:
                stats["rejected"] += 1
                break
            stats["accepted"] += 1
        stats["accept_hist"][j - a - (0 if ok else 1)] += 1
        a = j + 1
    stats["parallel_efficiency"] = N / stats["target_calls"]
    return x, stats
