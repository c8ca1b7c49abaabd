"""CUDA-graph replay of generation steps (plumbing only: every step still runs in the library's
kernels).  One launch of the step kernel costs the host ~17 us from Python; for the small
workloads (a few MB of cache) that is twice the kernel's own time, and a captured graph replays
the same launches at 8-11 us each.

The step calls are asynchronous, keep no host-side state and read their counters from device
memory, so a captured sequence stays valid as the cache fills and evicts.
"""
from __future__ import annotations

import torch

from . import binding as a2sf


class GraphedSteps:
    """``steps`` consecutive generation steps on one cache, captured once and replayed.

    q, k_new, v_new: device tensors [steps, B, H, d] that the caller refills before each replay;
    out [steps, B, H, d] and evicted [steps, B, H] int32 receive the results.  Step t of a replay
    sees the cache as step t-1 left it, exactly as with single calls.
    """

    def __init__(self, cache: a2sf.Cache, alpha: float, q, k_new, v_new, out=None, evicted=None):
        steps, B, H, d = q.shape
        assert k_new.shape == q.shape and v_new.shape == q.shape
        self.cache, self.alpha = cache, alpha
        self.q, self.k_new, self.v_new = q, k_new, v_new
        self.out = out if out is not None else torch.empty_like(q)
        self.evicted = (evicted if evicted is not None
                        else torch.empty((steps, B, H), dtype=torch.int32, device=q.device))
        # the first step call on a device sets kernel attributes: it must run outside a capture.
        # It would also change the cache, so it runs on a scratch cache of the same shape.
        scratch = a2sf.Cache(cache.p, q.device)
        scratch.a2sf_decode_step(alpha, q[0], k_new[0], v_new[0], self.out[0], self.evicted[0])
        torch.cuda.current_stream().synchronize()
        scratch.close()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            for t in range(steps):
                cache.a2sf_decode_step(alpha, q[t], k_new[t], v_new[t], self.out[t], self.evicted[t])

    def replay(self):
        """Runs the captured steps on the current contents of q, k_new, v_new."""
        self.graph.replay()
        return self.out, self.evicted
