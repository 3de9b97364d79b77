"""Helpers shared by the GPU parity tests: device upload of the seeded inputs and tolerance rules."""
import numpy as np
import torch

from paper_2601_08273_b200 import workloads as W


def dev(x: np.ndarray, dtype: str = None) -> torch.Tensor:
    """Upload a numpy array; with dtype="bf16" the fp32 values (already bf16-representable) become bf16."""
    if dtype == "bf16":
        bits = W.to_bf16_bits(x)
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def host(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy()
    return t.cpu().numpy()


def paged_cache(binding, k, v, lens, dtype, shuffle_seed=None, spare=0, fill=0.0, caps=None):
    """Logical k, v [B][T][H][D] -> (KVCache, page_table ndarray, n_pool)."""
    rng = None if shuffle_seed is None else np.random.default_rng(shuffle_seed)
    caps = lens if caps is None else caps
    table, n_pool = W.make_page_table(caps, rng, spare_pages=spare)
    kp = dev(W.pack_paged(k, lens, table, n_pool, fill=fill), dtype)
    vp = dev(W.pack_paged(v, lens, table, n_pool, fill=fill), dtype)
    if shuffle_seed is None and len(lens) == 1:
        return binding.KVCache(kp, vp, None, table.shape[1]), table, n_pool
    return binding.KVCache(kp, vp, dev(table)), table, n_pool


def assert_close(got: np.ndarray, ref: np.ndarray, tol: float, what: str = ""):
    """|got - ref| <= tol * (1 + |ref|) element by element."""
    err = np.abs(got.astype(np.float64) - ref)
    bound = tol * (1.0 + np.abs(ref))
    bad = err > bound
    assert not bad.any(), "%s: %d / %d elements off, worst |err| %.3e at %s (ref %.5f got %.5f)" % (
        what, bad.sum(), bad.size, err.max(), np.unravel_index(err.argmax(), err.shape),
        ref.reshape(-1)[err.argmax()], got.reshape(-1)[err.argmax()])


TOL = {"fp32": 1e-5, "bf16": 2e-2}
