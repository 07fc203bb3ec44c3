"""Helpers shared by the tests, the smoke check and the bench: move a synthetic workload to the device,
register its models and run one mixed batch through the C-ABI.  Marshalling only."""
from __future__ import annotations

from typing import List, Sequence

import numpy as np
import torch

from . import binding as mt


def bf16_bits_to_device(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def register_models(models: Sequence) -> List[int]:
    return [mt.mt_register_model(m) for m in models]


def run_batch(model_ids: np.ndarray, inputs_bits: np.ndarray, out_elems: int) -> np.ndarray:
    """One mt_infer on device copies of the given host arrays; returns fp32 [n, out_elems] as numpy."""
    n = int(model_ids.shape[0])
    x = bf16_bits_to_device(inputs_bits.reshape(n, -1))
    ids = torch.from_numpy(np.ascontiguousarray(model_ids, dtype=np.int32)).cuda()
    out = torch.full((n, out_elems), float("nan"), dtype=torch.float32, device="cuda")
    mt.mt_infer(x, ids, n, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def scaled_error(got: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """|gpu - oracle| / max(1, |oracle|) per element (the parity metric; tolerance 2e-2)."""
    return np.abs(got.astype(np.float64) - ref) / np.maximum(1.0, np.abs(ref))
