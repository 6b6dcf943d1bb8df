"""Shared pieces of the GPU parity tests: run a DecodeSpec through the C-ABI, compare with
the fp64 oracle under the stated tolerance."""
import numpy as np
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl

# Tolerance.  Decode (pa_decode and every entry point built on it): the stated one for bf16
# inputs with fp32 accumulation -- element-wise |gpu - ref| <= 1e-2 and, per (sequence, head)
# row, max_d |gpu - ref| <= 2e-2 * max_d |ref|.  The decode kernel hands each softmax weight to
# the tensor core as two bf16 numbers (value and remainder), so its un-rounded result is the
# exact one to about 1e-5 and what remains is the rounding of the bf16 output itself.  The
# tests therefore hold decode to the tighter, element-wise
#     |gpu - ref|  <=  half a bf16 spacing at |ref|  +  5e-4,
# which is below 1e-2 for every |ref| < 4 (7.8e-3 + 5e-4 at most).  From |ref| = 4 on, half a
# spacing alone is 1.56e-2: no bf16 output can promise 1e-2 there, and the bound above is what
# the tests require instead (such elements are counted in the tally).
#
# Prefill (pa_prefill, pa_prefill_split) has no stated tolerance of its own; its bound follows
# from its arithmetic and equals the decode bound except on rare elements.  With w_t the softmax
# weights of a row, the kernel computes sum_t bf16(w_t) V_t (the weights are a tensor-core operand)
# over a row sum of the unrounded weights, then rounds the result to bf16:
#     |gpu - ref|  <=  half a bf16 spacing at |ref|        (rounding of the result)
#                    + 2^-8 * sum_t w_t |V_t|               (rounding of each weight)
#                    + 1e-3                                 (fp32 sums, approximated exponentials)
# bf16 keeps 8 significant bits, so rounding to it moves a value by up to 2^-8 of itself (the
# unit roundoff; half a spacing is 2^-8 of the power of two below the value).  The middle term
# is the attention output over |V| and comes from the same oracle.  Where that total exceeds
# 1e-2 it replaces 1e-2 (`amended`): a row whose softmax is one-hot on an element of V of
# magnitude 2.5 may be off by 7.8e-3 + 9.8e-3.  It takes an output of magnitude above 1, i.e. a
# softmax concentrated on a few extreme elements of V, for the total to pass 1e-2.  The tally
# below counts the elements that ever use it.  The row-normalised 2e-2 bound is the same for
# both.
ABS_TOL = 1e-2
REL_TOL = 2e-2
DECODE_SLACK = 5e-4     # decode: what the result may differ by before its rounding to bf16
GUARD = 4096            # guard elements on each side of a test's output buffer
GUARD_BITS = 0x7A5A     # their content (int16 view)

# running totals over every assert_parity call of the process (printed at the end of the run)
TALLY = {"calls": 0, "elements": 0, "amended_calls": 0, "amended_elements": 0,
         "decode_elements": 0, "decode_over_abs_tol": 0, "decode_over_min_ref": float("inf"),
         "over_abs_tol": 0, "over_abs_tol_min_ref": float("inf"), "over_abs_tol_max_err": 0.0,
         "over_abs_tol_where": []}


def half_spacing(ref: np.ndarray) -> np.ndarray:
    """Half the distance between neighbouring bf16 numbers (8 significant bits) at |ref|."""
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 8)


def decode_bound(ref: np.ndarray) -> np.ndarray:
    """Element-wise decode bound: the output's own rounding plus DECODE_SLACK."""
    return half_spacing(ref) + DECODE_SLACK


def amended_bound(ref: np.ndarray, abs_ref: np.ndarray) -> np.ndarray:
    """Element-wise prefill bound: max(1e-2, half spacing at |ref| + 2^-8 abs_ref + 1e-3), where
    abs_ref is the oracle's output for the same inputs with V replaced by |V|."""
    return np.maximum(ABS_TOL, half_spacing(ref) + abs_ref * 2.0 ** -8 + 1e-3)


def abs_bits(v_bits: np.ndarray) -> np.ndarray:
    """|V| on bf16 bit patterns (sign bit cleared; NaN tails stay NaN and stay masked)."""
    return v_bits & np.uint16(0x7FFF)


def prefill_ref(q, k, v, tables, ctx, cu, scale):
    """(oracle output, thunk returning the oracle output over |V|) for a prefill comparison."""
    ref = oracle.pa_prefill(q, k, v, tables, ctx, cu, scale)
    return ref, (lambda: oracle.pa_prefill(q, k, abs_bits(v), tables, ctx, cu, scale))


def assert_parity(gpu: np.ndarray, ref: np.ndarray, what: str = "", abs_tol: float = None,
                  amended=None):
    """Compare a GPU result with the oracle.  With neither `abs_tol` nor `amended` the decode
    bound applies.  `amended` (prefill results only) is a callable returning the oracle's output
    over |V|, shaped like `ref`; it is evaluated only when some element exceeds the plain bound.
    An explicit `abs_tol` is a plain element-wise bound (comparisons between two GPU results)."""
    gpu = np.asarray(gpu, dtype=np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.isfinite(gpu).all(), f"{what}: non-finite output"
    err = np.abs(gpu - ref)
    over = err > ABS_TOL
    TALLY["calls"] += 1
    TALLY["elements"] += err.size
    if abs_tol is not None:
        bound = np.full_like(err, abs_tol)
    elif amended is None:
        bound = decode_bound(ref)
        TALLY["decode_elements"] += err.size
        if over.any():
            TALLY["decode_over_abs_tol"] += int(over.sum())
            TALLY["decode_over_min_ref"] = min(TALLY["decode_over_min_ref"],
                                               float(np.abs(ref[over]).min()))
    else:
        bound = np.full_like(err, ABS_TOL)
        TALLY["amended_calls"] += 1
        TALLY["amended_elements"] += err.size
        if over.any():
            TALLY["over_abs_tol"] += int(over.sum())
            TALLY["over_abs_tol_min_ref"] = min(TALLY["over_abs_tol_min_ref"],
                                                float(np.abs(ref[over]).min()))
            TALLY["over_abs_tol_max_err"] = max(TALLY["over_abs_tol_max_err"], float(err[over].max()))
            TALLY["over_abs_tol_where"].append(f"{what}: {int(over.sum())} of {err.size}")
            abs_ref = np.asarray(amended(), dtype=np.float64)
            assert abs_ref.shape == ref.shape
            bound = amended_bound(ref, abs_ref)
    worst = np.unravel_index(np.argmax(err - bound), err.shape) if err.size else ()
    assert (err <= bound).all(), (f"{what}: abs err {err[worst]:.3e} at ref {ref[worst]:.4f} "
                                  f"(bound {bound[worst]:.3e})")
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
