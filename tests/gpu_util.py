"""Helpers shared by the GPU parity tests: upload of the seeded host buffers, tolerance check."""
import numpy as np
import torch

from paper_2607_28418_b200 import synth

REL_TOL = 2e-2  # max |err| <= REL_TOL * max |ref|  (bf16 inputs, fp32 accumulation)


def to_dev(a: np.ndarray, dtype: str) -> torch.Tensor:
    """float32 host array -> CUDA tensor of the workload dtype (exact for bf16-rounded inputs)."""
    from paper_2607_28418_b200 import binding
    return binding.upload(a, dtype)


def bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int32)).cuda()


def bits_to_host(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def assert_close(y_gpu: torch.Tensor, y_ref: np.ndarray, what: str = "", rel: float = REL_TOL):
    got = y_gpu.float().cpu().numpy().astype(np.float64)
    scale = float(np.abs(y_ref).max())
    err = float(np.abs(got - y_ref).max()) if got.size else 0.0
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    assert err <= rel * scale + 1e-30, f"{what}: max|err| {err:.4e} > {rel} * max|ref| {scale:.4e}"
    return err / scale if scale > 0 else 0.0


def meta_to_dev(meta: dict) -> dict:
    """Oracle reorder output -> device tensors in the layout wide_ffn expects."""
    n_tiles, NG = meta["tile_map"].shape
    wl = np.full((max(n_tiles * NG, 1), 2), -1, dtype=np.int32)
    wl[: meta["n_work"]] = meta["work_list"]
    return {
        "perm": torch.from_numpy(meta["perm"]).cuda(),
        "counts": torch.from_numpy(meta["counts"]).cuda(),
        "work_list": torch.from_numpy(wl).cuda(),
        "n_work": torch.tensor([meta["n_work"]], dtype=torch.int32).cuda(),
        "offsets": torch.from_numpy(meta["offsets"]).cuda(),
        "token_order": torch.from_numpy(meta["token_order"]).cuda(),
        "token_rank": torch.from_numpy(meta["token_rank"]).cuda(),
    }


def ffn_ref_rows(case: dict, mask: np.ndarray, group: int, chunk: int = 1024) -> np.ndarray:
    """The oracle's FFN over EVERY token row, computed a block of rows at a time (an output row
    depends only on its own token and mask row, Eq. 3) so that the fp64 hidden activation of one
    block, not of the whole batch, is alive at any moment."""
    from oracle import wide_oracle as wo
    T = case["x"].shape[0]
    out = np.empty((T, case["w_down"].shape[0]), dtype=np.float64)
    for r0 in range(0, T, chunk):
        r1 = min(T, r0 + chunk)
        out[r0:r1] = wo.ffn(case["x"][r0:r1], case["w_gate"], case["w_up"], case["w_down"], mask[r0:r1], group)
    return out


def assert_all_rows_close(y_gpu: torch.Tensor, y_ref: np.ndarray, what: str, rel: float = REL_TOL) -> float:
    """Element-by-element comparison of the whole output: max|err| <= rel * max|ref|."""
    got = y_gpu.float().cpu().numpy()
    assert got.shape == y_ref.shape, f"{what}: shape {got.shape} vs {y_ref.shape}"
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    scale = float(np.abs(y_ref).max())
    err = 0.0
    for r0 in range(0, got.shape[0], 2048):       # blockwise: no second full-size fp64 temporary
        err = max(err, float(np.abs(got[r0:r0 + 2048].astype(np.float64) - y_ref[r0:r0 + 2048]).max()))
    assert err <= rel * scale + 1e-30, f"{what}: max|err| {err:.4e} > {rel} * max|ref| {scale:.4e}"
    return err / scale if scale > 0 else 0.0
