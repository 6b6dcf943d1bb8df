"""Shared pieces of the GPU parity tests: run a DecodeSpec through the C-ABI, compare with
the fp64 oracle under the stated tolerance."""
import numpy as np
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl

# Tolerance for bf16 inputs with fp32 accumulation: element-wise |gpu - ref| <= 1e-2 and,
# per (sequence, head) row, max_d |gpu - ref| <= 2e-2 * max_d |ref|.  The output is bf16:
# from 2 upwards its values are 2^-6 apart (2^-5 from 4), so rounding the result alone takes
# up to 7.8e-3 (1.6e-2) and the bf16 rounding of the softmax weights adds up to 2^-9 of the
# magnitude; there the element-wise bound is one spacing of bf16 at |ref| instead of 1e-2.
# Outputs that large need a softmax that is nearly one-hot on an extreme element of V.
ABS_TOL = 1e-2
REL_TOL = 2e-2
GUARD = 4096            # guard elements on each side of a test's output buffer
GUARD_BITS = 0x7A5A     # their content (int16 view)


def assert_parity(gpu: np.ndarray, ref: np.ndarray, what: str = "", abs_tol: float = ABS_TOL):
    gpu = np.asarray(gpu, dtype=np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.isfinite(gpu).all(), f"{what}: non-finite output"
    err = np.abs(gpu - ref)
    spacing = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 7)   # of bf16 at |ref|
    excess = err - np.maximum(abs_tol, np.where(np.abs(ref) >= 2.0, spacing, 0.0))
    assert excess.max(initial=-1.0) <= 0.0, f"{what}: abs err {err.max():.3e}"
    row_err = err.reshape(-1, err.shape[-1]).max(axis=1)
    row_ref = np.abs(ref).reshape(-1, ref.shape[-1]).max(axis=1)
    rel = row_err / np.maximum(row_ref, 1e-30)
    nz = row_ref > 0
    assert (rel[nz] <= REL_TOL).all(), f"{what}: row-normalised rel err {rel[nz].max():.3e}"
    assert (row_err[~nz] == 0).all(), f"{what}: non-zero output where the oracle is zero"
    return float(rel[nz].max(initial=0.0))


def bits_to_torch(bits: np.ndarray, device="cuda"):
    return torch.from_numpy(bits.view(np.int16).copy()).to(device).view(torch.bfloat16)


def torch_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


class GpuDecode:
    """Device buffers for one spec plus a `run` that calls pa_decode through the binding."""

    def __init__(self, spec, q_bits=None, k_bits=None, v_bits=None, tables=None, lens=None,
                 max_tokens=None, partition_tokens=0):
        self.spec = spec
        dev = "cuda"
        self.q = bits_to_torch(q_bits) if q_bits is not None else wl.q_torch(spec, dev)
        if k_bits is not None:
            self.k, self.v = bits_to_torch(k_bits), bits_to_torch(v_bits)
        else:
            self.k, self.v = wl.pools_torch(spec, dev)
        self.tables = torch.from_numpy(np.ascontiguousarray(
            spec.block_tables if tables is None else tables)).to(dev)
        self.lens = torch.from_numpy(np.ascontiguousarray(
            spec.seq_lens if lens is None else lens).astype(np.int32)).to(dev)
        # output and workspace sit between guard zones holding a bit pattern: with no memory
        # checker available, a kernel that writes outside its buffers is caught here
        n_out = self.q.numel()
        self._out_store = torch.full((n_out + 2 * GUARD,), GUARD_BITS, dtype=torch.int16, device=dev)
        self.out = self._out_store[GUARD:GUARD + n_out].view(torch.bfloat16).view(self.q.shape)
        self.out.fill_(float("nan"))
        shape = api.shape_of(self.k, self.q.shape[1])
        tot = int(max_tokens if max_tokens is not None else
                  self.tables.shape[0] * self.tables.shape[1] * 16)
        nbytes = api.pa_workspace_bytes(shape, self.q.shape[0], tot, partition_tokens)
        nbytes = (nbytes + 255) & ~255
        self._ws_store = torch.full((nbytes + 2 * 4096,), 0x5A, dtype=torch.uint8, device=dev)
        self.ws = self._ws_store[4096:4096 + nbytes]
        assert self.ws.data_ptr() % 256 == 0
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.partition_tokens = partition_tokens

    def run(self, scale=None, **kw):
        self.out.fill_(float("nan"))
        kw.setdefault("partition_tokens", self.partition_tokens)
        api.pa_decode(self.q, self.k, self.v, self.tables, self.lens,
                      self.spec.scale if scale is None else scale, self.out, self.ws,
                      dev_status=self.status, **kw)
        torch.cuda.synchronize()
        self.check_guards()
        return self.out

    def check_guards(self):
        n = self.q.numel()
        assert bool((self._out_store[:GUARD] == GUARD_BITS).all()), "write before the output"
        assert bool((self._out_store[GUARD + n:] == GUARD_BITS).all()), "write past the output"
        assert bool((self._ws_store[:4096] == 0x5A).all()), "write before the workspace"
        assert bool((self._ws_store[4096 + self.ws.numel():] == 0x5A).all()), "write past the workspace"

    def plan_header(self):
        return self.ws[:64 * 4].view(torch.int32).cpu().numpy()


def oracle_for(spec, q_bits, k_bits, v_bits, tables=None, lens=None, scale=None):
    return oracle.pa_decode(q_bits, k_bits, v_bits,
                            spec.block_tables if tables is None else tables,
                            spec.seq_lens if lens is None else lens,
                            spec.scale if scale is None else scale)
