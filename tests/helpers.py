"""Shared pieces of the GPU parity tests: run the C-ABI library on seeded inputs and
compare with the CPU oracle."""
import numpy as np

REL_TOL = 5e-3          # relative Frobenius error allowed per bf16-in / fp32-accumulate GEMM output


def rel_fro(gpu_f64: np.ndarray, ref: np.ndarray) -> float:
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(gpu_f64 - ref) / (den if den > 0 else 1.0))


# Elementwise bound beside the per-tensor norm.  One fp32 -> bf16 rounding moves an element by at
# most half a unit in the last place, i.e. 2^-8 of its magnitude; what the fp32 accumulation and a
# bf16-rounded adapter operand add is independent of the element's own size, so it is allowed
# relative to the tensor's root mean square: 2^-9 for outputs rounded once (measured: fp32
# accumulation ~1e-6, the adapter term's bf16 T ~1e-4 of the rms), 2^-6 for the gradients that are
# sums over a bf16-rounded intermediate (dL over dT, dR over T: a Gaussian error of ~1.7e-3 rms per
# element, whose largest value over a million elements is ~5 sigma).  A single wrong element (a
# dropped k-block, a wrong metadata code) is off by a large fraction of the rms and fails this
# where the Frobenius norm of a big tensor would hide it.
ELEM_REL = 2.0 ** -8
ELEM_RMS = {1: 2.0 ** -9, 2: 2.0 ** -6}


def parity_error(gpu_f64: np.ndarray, ref: np.ndarray, roundings: int = 1) -> float:
    """Relative Frobenius error of a GPU output against the oracle; raises when any single
    element is further off than bf16 rounding (plus the slack above) explains."""
    gpu_f64, ref = np.asarray(gpu_f64, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    assert gpu_f64.shape == ref.shape, (gpu_f64.shape, ref.shape)
    rms = float(np.sqrt(np.mean(ref * ref))) if ref.size else 0.0
    bound = ELEM_REL * np.abs(ref) + ELEM_RMS[roundings] * rms
    excess = np.abs(gpu_f64 - ref) - bound
    bad = int(np.count_nonzero(~(excess <= 0)))          # NaN counts as bad
    if bad:
        worst = np.unravel_index(int(np.nanargmax(np.where(np.isnan(excess), np.inf, excess))), ref.shape)
        raise AssertionError(f"{bad} of {ref.size} elements outside the elementwise bound; worst at {worst}: "
                             f"gpu {gpu_f64[worst]!r} oracle {ref[worst]!r} bound {bound[worst]!r} (rms {rms!r})")
    return rel_fro(gpu_f64, ref)


def to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


class GpuLayer:
    """Device-side state of one SLoPe layer driven through the C ABI."""

    def __init__(self, W_bits, device="cuda", fused_setup=False):
        import torch
        from paper_2608_24070_b200 import binding as B

        self.B = B
        self.torch = torch
        self.d_out, self.d_in = W_bits.shape
        self.W = B.bf16_from_bits(W_bits, device)
        self.Wc_vals, self.Wc_meta, self.mask1 = B.alloc_compressed(self.d_out, self.d_in, device)
        self.WTc_vals, self.WTc_meta, _ = B.alloc_compressed(self.d_in, self.d_out, device)
        self.mask2 = torch.empty_like(self.mask1)
        if fused_setup:      # both pruning passes in one launch
            B.slope_prune_24_double(self.W, self.Wc_vals, self.Wc_meta, self.mask1, self.WTc_vals, self.WTc_meta,
                                    self.mask2)
        else:
            B.slope_prune_24(self.W, self.Wc_vals, self.Wc_meta, self.mask1)
            B.slope_double_prune(self.W, self.mask1, self.WTc_vals, self.WTc_meta, self.mask2)

    def canonical(self, meta, rows, cols):
        out = self.torch.empty((rows, cols // 16), dtype=self.torch.int16, device=meta.device)
        self.B.slope_meta_to_canonical(meta, rows, cols, out)
        return out.cpu().numpy().view(np.uint16)

    def fwd(self, X, T=None, R=None):
        Y = self.torch.empty((X.shape[0], self.d_out), dtype=self.torch.bfloat16, device=X.device)
        self.B.slope_linear_fwd(X, self.Wc_vals, self.Wc_meta, self.d_out, Y, T, R)
        return Y

    def dx(self, dY, dT=None, L=None):
        dX = self.torch.empty((dY.shape[0], self.d_in), dtype=self.torch.bfloat16, device=dY.device)
        self.B.slope_linear_bwd_dx(dY, self.WTc_vals, self.WTc_meta, self.d_in, dX, dT, L)
        return dX

    def dw(self, dY, X):
        dWc = self.torch.empty((self.d_out, self.d_in // 2), dtype=self.torch.bfloat16, device=X.device)
        self.B.slope_linear_bwd_dw_masked(dY, X, self.mask1, dWc)
        return dWc

    def adapter_T(self, X, L):
        b, r = X.shape[0], L.shape[1]
        T = self.torch.empty((b, r), dtype=self.torch.bfloat16, device=X.device)
        self.B.slope_adapter_fwd_bwd(0, X, None, L, None, b, self.d_out, self.d_in, r, T=T)
        return T

    def adapter_bwd(self, X, dY, L, R, T):
        torch = self.torch
        b, r = X.shape[0], L.shape[1]
        dT = torch.empty((b, r), dtype=torch.bfloat16, device=X.device)
        dL = torch.empty((self.d_in, r), dtype=torch.bfloat16, device=X.device)
        dR = torch.empty((r, self.d_out), dtype=torch.bfloat16, device=X.device)
        ws = torch.empty(self.B.slope_adapter_workspace_bytes(b, self.d_out, self.d_in, r), dtype=torch.uint8,
                         device=X.device)
        self.B.slope_adapter_fwd_bwd(1, X, dY, L, R, b, self.d_out, self.d_in, r, T=T, dT=dT, dL=dL, dR=dR,
                                     workspace=ws)
        return dT, dL, dR

    def poll(self):
        st = self.B.slope_poll_status()
        assert st == 0, self.B.slope_status_string(st)


def check_selection(oracle, layer: GpuLayer, W_bits):
    """Bit-exact comparison of everything the two pruning passes write."""
    B = layer.B
    vals, nib, mask1 = oracle.prune24(W_bits)
    valsT, nibT, mask2 = oracle.double_prune(W_bits, mask1)
    layer.poll()
    assert np.array_equal(B.bits_from_bf16(layer.Wc_vals), vals), "first-pass values"
    assert np.array_equal(layer.mask1.cpu().numpy(), mask1), "first-pass mask"
    canon = oracle.pack_canonical(nib)
    assert np.array_equal(layer.Wc_meta.cpu().numpy(), oracle.canonical_to_hw(canon)), "first-pass metadata"
    assert np.array_equal(layer.canonical(layer.Wc_meta, layer.d_out, layer.d_in), canon), "canonical metadata"
    assert np.array_equal(B.bits_from_bf16(layer.WTc_vals), valsT), "second-pass values"
    assert np.array_equal(layer.mask2.cpu().numpy(), mask2), "second-pass mask"
    canonT = oracle.pack_canonical(nibT)
    assert np.array_equal(layer.WTc_meta.cpu().numpy(), oracle.canonical_to_hw(canonT)), "second-pass metadata"
    assert np.array_equal(layer.canonical(layer.WTc_meta, layer.d_in, layer.d_out), canonT)
    return mask1, mask2
