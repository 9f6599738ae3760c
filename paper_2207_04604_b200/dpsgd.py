"""Privacy-preserving D-PSGD (Algorithm 2) around the library's whole-round call.

Each iteration every user computes a local gradient, the users' current parameters go through
one private gradient update on the GPU (fixed-point encode, encrypt under the collective key,
neighbour sums, collective decryption), the decoded sums are divided by the closed-neighbourhood
size (the mixing weights E_ij = 1/|U_i| are applied after decryption) and the local SGD step
follows.  The model side (objective, gradient) is the caller's; this module owns only the
protocol plumbing, which makes the loss-free claim of Sec. 6 checkable: the result equals
plaintext D-PSGD run on the same fixed-point values bit for bit.
"""
import numpy as np
import torch

from . import workloads as wl


def to_fixed(w, clip):
    """fp32 parameters -> int32 fixed point (scale 2^10), clipped so that neighbour sums cannot wrap."""
    return wl.quantise(np.asarray(w, dtype=np.float32), clip)


def from_fixed(v):
    return np.asarray(v, dtype=np.float64) / wl.FIXED_POINT_SCALE


class PrivateDPSGD:
    """K users, parameter vectors of length H, closed neighbourhoods in CSR form."""

    def __init__(self, ctx, offsets, rows, param_len, chunk_cts=None):
        self.ctx = ctx
        self.K, self.n = ctx.num_parties, ctx.n
        self.offsets = np.asarray(offsets, dtype=np.uint32)
        self.rows = np.asarray(rows, dtype=np.uint32)
        self.H = int(param_len)
        self.C = -(-self.H // self.n)
        self.clip = ((ctx.t - 1) // 2) // self.K
        self.sizes = np.diff(self.offsets).astype(np.float64)[:, None]
        chunk = self.C if chunk_cts is None else chunk_cts
        self.ws = torch.empty(ctx.round_workspace_bytes(chunk), dtype=torch.uint8, device=ctx.device)
        self.values = torch.zeros((self.K, self.C, self.n), dtype=torch.int32, device=ctx.device)
        self.sums = torch.zeros_like(self.values)
        self.iteration = 0

    def mix(self, weights):
        """weights: float [K, H].  Returns the neighbourhood averages [K, H] computed under encryption."""
        fixed = np.zeros((self.K, self.C * self.n), dtype=np.int32)
        fixed[:, :self.H] = to_fixed(weights, self.clip)
        self.values.copy_(torch.from_numpy(fixed.reshape(self.K, self.C, self.n)))
        # every iteration uses fresh ciphertext indices, hence fresh randomness
        self.ctx.round_device(self.values, self.iteration * self.C, self.C, self.offsets, self.rows, self.sums,
                              self.ws)
        self.ctx.sync()
        self.iteration += 1
        total = self.sums.cpu().numpy().reshape(self.K, -1)[:, :self.H]
        return from_fixed(total) / self.sizes

    def step(self, weights, grads, lr):
        """One iteration of Algorithm 2: W_{k+1,i} = mix(W_k)_i - lr * grad_i."""
        return self.mix(weights) - lr * np.asarray(grads, dtype=np.float64)


def plaintext_mix(weights, offsets, rows, clip):
    """The same averaging on the same fixed-point values without encryption (Algorithm 1)."""
    fixed = to_fixed(weights, clip).astype(np.int64)
    out = np.stack([fixed[rows[offsets[i]:offsets[i + 1]]].sum(axis=0) for i in range(len(offsets) - 1)])
    return from_fixed(out) / np.diff(offsets).astype(np.float64)[:, None]
