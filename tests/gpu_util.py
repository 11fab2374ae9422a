"""Helpers shared by the GPU parity tests: moving seeded host arrays to the device, running the
oracle on the same arrays, and the tolerance checks stated by the task (bit-exact tables, fp32
scores within 1e-5 relative, bf16 outputs within 1e-2 relative Frobenius and 3e-2 max-abs)."""
import numpy as np
import torch

import oracle
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200.workloads import bf16_bits_to_f32, f32_to_bf16_bits


def dev_bf16(bits):
    return cwl.bf16_from_bits(bits)


def host_table(d):
    return oracle.ChunkTable(np.asarray(d["offsets"], np.int32), np.asarray(d["rank"], np.int32),
                             np.asarray(d["scale"], np.float32),
                             np.asarray(d.get("rung", np.zeros(len(d["rank"]))), np.int32),
                             np.asarray(d["flags"], np.int32), int(d["n_chunks"]))


def dev_table(d):
    return cwl.DeviceChunkTable.from_host(d["offsets"], d["rank"], d["scale"], d["flags"], d.get("rung"))


def table_dict(t: oracle.ChunkTable):
    return dict(offsets=t.offsets, rank=t.rank, scale=t.scale, rung=t.rung, flags=t.flags, n_chunks=t.n_chunks)


def y_to_f64(Y: torch.Tensor) -> np.ndarray:
    bits = Y.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return bf16_bits_to_f32(bits).astype(np.float64)


def check_output(y_gpu: np.ndarray, y_ref: np.ndarray):
    """Relative Frobenius <= 1e-2; every entry within 3e-2, or within one bf16 ulp of the rounded
    reference (half an ulp of bf16 alone exceeds 3e-2 once |y| >= 8).  Returns the figures."""
    diff = np.abs(y_gpu - y_ref)
    rel_fro = float(np.linalg.norm(y_gpu - y_ref) / max(np.linalg.norm(y_ref), 1e-30))
    ref_bf16 = bf16_bits_to_f32(f32_to_bf16_bits(y_ref.astype(np.float32))).astype(np.float64)
    ulp = np.maximum(np.abs(ref_bf16), 2.0 ** -126) * 2.0 ** -7
    within_ulp = np.abs(y_gpu - ref_bf16) <= ulp
    bad = (diff > 3e-2) & ~within_ulp
    assert rel_fro <= 1e-2, f"relative Frobenius error {rel_fro:.3e}"
    assert not bad.any(), f"{int(bad.sum())} entries off by more than 3e-2 and one bf16 ulp; max abs {diff.max():.3e}"
    return dict(rel_fro=rel_fro, max_abs=float(diff.max()), saved_by_ulp=int(((diff > 3e-2) & within_ulp).sum()))


def status_ok(status_word: torch.Tensor):
    assert int(status_word.item()) == 0, f"device status word {int(status_word.item()):#x}"
