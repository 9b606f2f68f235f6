"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from paper_2107_05377_b200 import synth


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 tensor on the GPU (same bits)."""
    return torch.from_numpy(bits.astype(np.int16)).view(torch.bfloat16).cuda()


def dev_bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def rand_bf16(seed: int, name: str, shape, std: float, mean: float = 0.0):
    """Seeded bf16 array: returns (bits uint16, exact float64 values)."""
    n = int(np.prod(shape))
    x = (mean + std * synth.standard_normal(seed, name, n)).astype(np.float32)
    bits = synth.f32_to_bf16_bits(x).reshape(shape)
    return bits, synth.bf16_bits_to_f64(bits)


def rel_l2(got: np.ndarray, want: np.ndarray) -> float:
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30))


_WEIGHT_CACHE = {}


def cached_weights(cfg, seed=0, random_affine=False):
    """(bf16-bit weights, packed blob, widened fp64 weights) - generated once per test session."""
    key = (cfg, seed, random_affine)
    if key not in _WEIGHT_CACHE:
        w = synth.make_weights(cfg, seed=seed, random_affine=random_affine)
        _WEIGHT_CACHE[key] = (w, synth.pack_weights(cfg, w), synth.widen(w))
    return _WEIGHT_CACHE[key]


def task_triples(cfg):
    """Task tuples for the oracle; token-level tasks carry their head kind as a fourth entry."""
    return [(t.fork_depth, t.branch_layers, t.num_classes) + ((1,) if t.token_level else ()) for t in cfg.tasks]


def dev_batch(batch):
    return (torch.from_numpy(batch.token_ids).cuda(), torch.from_numpy(batch.segment_ids).cuda(),
            torch.from_numpy(batch.lengths).cuda())
