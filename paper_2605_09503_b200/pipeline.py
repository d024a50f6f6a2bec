"""Sequencing of the C-ABI calls into the two halves of the method.  No arithmetic happens
here: every step is one entry point of libpq.so, all enqueued on the current stream without a
host round trip (the accept decision stays on the device and is consumed by pq_quant_weight).

  calibrate()    offline: statistics -> Eq. 9 candidates -> Eq. 3 errors -> Eq. 10 -> P^T W quantized
  QuantLinear    runtime: bf16 activations (already permuted) -> NVFP4 -> W4A4 GEMM -> bf16
  calibrate_h()  the same offline pass in the Hadamard-transformed basis (PermuQuant-H, App. D)
  QuantLinearH   runtime of PermuQuant-H: Hadamard + reordering + NVFP4 in one kernel, then the GEMM
"""
from dataclasses import dataclass

import torch

from . import binding as B

NVFP4 = (B.KIND_NVFP4, 4, 16)


@dataclass
class Calibration:
    """Everything the offline pass produces, all on the device."""
    sumsq_a: torch.Tensor      # fp64 [K]
    sumsq_w: torch.Tensor      # fp64 [K]
    amax_a: torch.Tensor       # fp32 [K]
    ts_x: torch.Tensor         # fp32 [1] static activation tensor scale
    ts_w: torch.Tensor         # fp32 [1]
    perms: torch.Tensor        # int32 [J+1, K] candidates, row j <-> alpha = j/J
    err_x: torch.Tensor        # fp64 [J+2, K/g], row 0 = original order
    err_w: torch.Tensor        # fp64 [J+2, K/g]
    lam: torch.Tensor          # fp64 [2]
    E: torch.Tensor            # fp64 [J+2]
    select: torch.Tensor       # int32 [2] = {best, accept}
    wq: torch.Tensor           # uint8 [N, K/2]
    sfw: torch.Tensor          # uint8, tensor-core layout
    rows_a: int

    def chosen_perm(self) -> torch.Tensor:
        """The order the acceptance rule kept (identity if rejected), as int64 indices."""
        best, accept = self.select.tolist()
        K = self.perms.shape[1]
        if accept:
            return self.perms[best - 1].long()
        return torch.arange(K, device=self.perms.device)


def calibrate(batches, Wt, fmt=NVFP4, J=5, tau=0.0, sf_layout=B.PQ_SF_TCGEN05) -> Calibration:
    """Offline pass over calibration batches (list of bf16 [T, K] device tensors) and the weight
    Wt (bf16 [N, K] device tensor).  `fmt` is the format whose error drives the acceptance rule."""
    dev = Wt.device
    N, K = Wt.shape
    group = 16 if fmt[0] == B.KIND_NVFP4 else fmt[2]
    Kg = K // group
    sumsq_a = torch.zeros(K, dtype=torch.float64, device=dev)
    sumsq_w = torch.zeros(K, dtype=torch.float64, device=dev)
    amax_a = torch.zeros(K, dtype=torch.float32, device=dev)
    amax_w = torch.zeros(K, dtype=torch.float32, device=dev)
    rows_a = 0
    max_rows = max([b.shape[0] for b in batches] + [N])
    ws = B.workspace(B.OP_GROUP_ERROR, max_rows, K, 0, J + 1)     # large enough for every step below
    ws_stats = B.workspace(B.OP_CALIB_STATS, max_rows, K)
    for x in batches:
        B.pq_calib_stats(x, sumsq_a, amax_a, ws_stats)
        rows_a += x.shape[0]
    B.pq_calib_stats(Wt, sumsq_w, amax_w, ws_stats)
    ts_x = torch.empty(1, dtype=torch.float32, device=dev)
    ts_w_err = torch.empty(1, dtype=torch.float32, device=dev)
    B.pq_tensor_scale(amax_a, ts_x)
    B.pq_tensor_scale(amax_w, ts_w_err)

    perms = torch.empty(J + 1, K, dtype=torch.int32, device=dev)
    B.pq_select_perm(sumsq_a, rows_a, sumsq_w, N, J, perms, B.workspace(B.OP_SELECT_PERM, 0, K, 0, J + 1))

    err_x = torch.zeros(J + 2, Kg, dtype=torch.float64, device=dev)
    err_w = torch.zeros(J + 2, Kg, dtype=torch.float64, device=dev)
    for x in batches:
        B.pq_group_error(x, fmt, ts_x, None, err_x[0:1], ws)
        B.pq_group_error(x, fmt, ts_x, perms, err_x[1:], ws)
    B.pq_group_error(Wt, fmt, ts_w_err, None, err_w[0:1], ws)
    B.pq_group_error(Wt, fmt, ts_w_err, perms, err_w[1:], ws)

    lam = torch.empty(2, dtype=torch.float64, device=dev)
    B.pq_error_weights(sumsq_a, sumsq_w, lam)
    select = torch.zeros(2, dtype=torch.int32, device=dev)
    E = torch.empty(J + 2, dtype=torch.float64, device=dev)
    B.pq_accept(err_x, err_w, lam, tau, select[0:1], select[1:2], E)

    wq = torch.empty(N, K // 2, dtype=torch.uint8, device=dev)
    sfw = torch.empty(B.sf_bytes(N, K, sf_layout), dtype=torch.uint8, device=dev)
    ts_w = torch.empty(1, dtype=torch.float32, device=dev)
    B.pq_quant_weight(Wt, perms, select, wq, sfw, sf_layout, ts_w, B.workspace(B.OP_QUANT_WEIGHT, N, K))
    return Calibration(sumsq_a, sumsq_w, amax_a, ts_x, ts_w, perms, err_x, err_w, lam, E, select, wq, sfw, rows_a)


def calibrate_h(batches, Wt, fmt=NVFP4, J=5, tau=0.0):
    """PermuQuant-H (App. D): the representation that is quantized is x H, so statistics, candidate
    orders, errors and the acceptance rule are all taken on the transformed calibration batches and on
    the transformed weight rows Wt H (the product is unchanged: (x H)(Wt H)^T = x Wt^T).  Returns the
    Calibration of the transformed layer; its chosen order is applied AFTER the transform at run time."""
    def transformed(t):
        out = torch.empty(t.shape[0], t.shape[1], dtype=torch.bfloat16, device=t.device)
        B.pq_hadamard_quant_nvfp4(t, None, None, None, None, B.PQ_SF_LINEAR, out)
        return out

    return calibrate([transformed(x) for x in batches], transformed(Wt), fmt=fmt, J=J, tau=tau)


def select_by_output_error(batches, refs, Wt, perms, ts_x, tau=0.0):
    """The acceptance rule of Eq. 10 with E read on the layer's output (Sec. 3.3): for the original
    order and every candidate row of `perms` (int32 [P, K]) quantize W and the calibration batches in
    that order, run the W4A4 GEMM and accumulate the squared distance to the unquantized outputs
    `refs` (fp32 [T, N] per batch, from any GEMM the caller trusts).  Returns (E fp64 [P+1], select
    int32 [2] = {best, accept}), both on the device; `select` is what pq_quant_weight consumes."""
    dev = Wt.device
    N, K = Wt.shape
    P = perms.shape[0]
    max_rows = max(b.shape[0] for b in batches)
    err = torch.zeros(P + 1, N, dtype=torch.float64, device=dev)
    wq = torch.empty(N, K // 2, dtype=torch.uint8, device=dev)
    sfw = torch.empty(B.sf_bytes(N, K, B.PQ_SF_TCGEN05), dtype=torch.uint8, device=dev)
    ts_w = torch.empty(1, dtype=torch.float32, device=dev)
    xq = torch.empty(max_rows, K // 2, dtype=torch.uint8, device=dev)
    sfx = torch.empty(B.sf_bytes(max_rows, K, B.PQ_SF_TCGEN05), dtype=torch.uint8, device=dev)
    Y = torch.empty(max_rows, N, dtype=torch.bfloat16, device=dev)
    ws_w = B.workspace(B.OP_QUANT_WEIGHT, N, K)
    ws_g = B.workspace(B.OP_GEMM, max_rows, K, N)
    ws_e = B.workspace(B.OP_OUTPUT_ERROR, max_rows, N)
    for p in range(P + 1):
        order = None if p == 0 else perms[p - 1]
        B.pq_quant_weight(Wt, order, None, wq, sfw, B.PQ_SF_TCGEN05, ts_w, ws_w)
        for x, ref in zip(batches, refs):
            T = x.shape[0]
            B.pq_quant_act_nvfp4_perm(x, order, ts_x, xq[:T], sfx, B.PQ_SF_TCGEN05)
            B.pq_gemm_w4a4(xq[:T], sfx, ts_x, wq, sfw, ts_w, Y[:T], ws_g)
            B.pq_output_error(ref, Y[:T], err[p], ws_e)
    select = torch.zeros(2, dtype=torch.int32, device=dev)
    E = torch.empty(P + 1, dtype=torch.float64, device=dev)
    B.pq_accept(err, torch.zeros_like(err), None, tau, select[0:1], select[1:2], E)
    return E, select


class QuantLinear:
    """Runtime half: holds the quantized weight and the intermediates of one layer."""

    def __init__(self, wq, sfw, ts_w, ts_x, M_max):
        self.wq, self.sfw, self.ts_w, self.ts_x = wq, sfw, ts_w, ts_x
        self.N, self.K = wq.shape[0], wq.shape[1] * 2
        dev = wq.device
        self.xq = torch.empty(M_max, self.K // 2, dtype=torch.uint8, device=dev)
        self.sfx = torch.empty(B.sf_bytes(M_max, self.K, B.PQ_SF_TCGEN05), dtype=torch.uint8, device=dev)
        self.ws = B.workspace(B.OP_GEMM, M_max, self.K, self.N)
        self.M_max = M_max
        self._sets = []          # further (xq, sfx) pairs for forward_batches

    def __call__(self, X, Y=None):
        M = X.shape[0]
        assert M <= self.M_max and X.shape[1] == self.K
        if Y is None:
            Y = torch.empty(M, self.N, dtype=torch.bfloat16, device=X.device)
        B.pq_linear_w4a4(X, self.ts_x, self.xq[:M], self.sfx, self.wq, self.sfw, self.ts_w, Y, self.ws)
        return Y

    def forward_batches(self, Xs, Ys, n_sets=4):
        """Independent batches through the layer, the quantizer of the next batches overlapped with
        the GEMM of the current one (pq_linear_w4a4_batched).  Extra sets of intermediates are kept."""
        M = Xs[0].shape[0]
        assert M <= self.M_max
        while len(self._sets) < n_sets:
            self._sets.append((torch.empty_like(self.xq), torch.empty_like(self.sfx)))
        xqs = [self.xq[:M]] + [a[:M] for a, _ in self._sets[:n_sets - 1]]
        sfxs = [self.sfx] + [b for _, b in self._sets[:n_sets - 1]]
        B.pq_linear_w4a4_batched(Xs, self.ts_x, xqs, sfxs, self.wq, self.sfw, self.ts_w, Ys, self.ws)
        return Ys

    def check(self):
        """Synchronise and raise if a bounded device-side wait expired."""
        code = B.pq_device_status(self.ws)
        if code != B.PQ_OK:
            raise B.PqError("pq_gemm_w4a4 (device)", code, B.status_string(code))


class QuantLinearH(QuantLinear):
    """Runtime half of PermuQuant-H: activations arrive in their ORIGINAL basis and order; one kernel
    applies the Hadamard transform, reads the transformed channels in the calibrated order and
    quantizes them (pq_hadamard_quant_nvfp4), then the W4A4 GEMM runs against the weight quantized by
    calibrate_h."""

    def __init__(self, wq, sfw, ts_w, ts_x, M_max, order):
        super().__init__(wq, sfw, ts_w, ts_x, M_max)
        self.order = None if order is None else order.to(torch.int32).contiguous()

    def __call__(self, X, Y=None):
        M = X.shape[0]
        assert M <= self.M_max and X.shape[1] == self.K
        if Y is None:
            Y = torch.empty(M, self.N, dtype=torch.bfloat16, device=X.device)
        B.pq_hadamard_quant_nvfp4(X, self.order, self.ts_x, self.xq[:M], self.sfx, B.PQ_SF_TCGEN05)
        B.pq_gemm_w4a4(self.xq[:M], self.sfx, self.ts_x, self.wq, self.sfw, self.ts_w, Y, self.ws)
        return Y
