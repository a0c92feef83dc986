"""Shared test helpers: upload seeded inputs, call the C ABI through the binding, error metrics."""
import numpy as np

from paper_2604_26294_b200 import inputs as inp


def bf16_tensor(bits: np.ndarray, device="cuda"):
    import torch

    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


def tensor_to_f64(t) -> np.ndarray:
    import torch

    if t.dtype == torch.bfloat16:
        return inp.bf16_bits_to_f64(t.view(torch.int16).cpu().numpy().view(np.uint16))
    return t.double().cpu().numpy()


def rel_fro(a: np.ndarray, ref: np.ndarray) -> float:
    return float(np.linalg.norm(a - ref) / max(np.linalg.norm(ref), 1e-300))


# Bound on worst_row_error() in the parity tests.  One bf16 rounding moves an element by at most 2^-9 of its own
# magnitude, and the largest element of a row of a few thousand roughly normal values is 4-5 row-RMS, which gives
# about 0.01; the rounding of the intermediate adds about as much again.  Measured over the whole GPU suite (the
# terminal summary prints it): largest value 0.022.  0.05 keeps a factor of two over that and is still far below
# what one wrong tile row (error of the order of 1 row-RMS) would produce.
TOL_ROW = 0.05

OBSERVED_ROW_ERRORS: list[float] = []


def worst_row_error(a: np.ndarray, ref: np.ndarray) -> float:
    """max over rows of max|a-ref| / rms(ref row): a bad patch cannot hide in a Frobenius norm."""
    rms = np.sqrt(np.mean(ref * ref, axis=1)) + 1e-30
    v = float(np.max(np.max(np.abs(a - ref), axis=1) / rms))
    OBSERVED_ROW_ERRORS.append(v)
    return v


class DeviceProblem:
    """Inputs of one seeded problem resident on the GPU in the library's layouts."""

    def __init__(self, S, H, F, D, seed=0, with_dy=False, host=None, options=None):
        import torch

        self.S, self.H, self.F, self.D = S, H, F, D
        self.options = dict(options or {})       # fields of tsp_mlp_options_t for the plans this problem creates
        self.host = host if host is not None else inp.make_inputs(S, H, F, seed=seed, with_dy=with_dy)
        h = self.host
        self.X = bf16_tensor(h.X)
        self.Wg = bf16_tensor(inp.shard_columns(h.Wg, D))
        self.Wu = bf16_tensor(inp.shard_columns(h.Wu, D))
        self.Wd = bf16_tensor(inp.shard_rows(h.Wd, D))
        self.dY = bf16_tensor(h.dY) if h.dY is not None else None
        self.Y = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")

    def forward(self, act=None):
        """Run tsp_mlp_forward through the binding; returns Y (torch bf16 on the GPU)."""
        import torch

        from paper_2604_26294_b200 import binding as b

        plan = b.tsp_mlp_plan_ex(self.H, self.F, self.D, **self.options)
        try:
            if act is not None:
                b.tsp_mlp_set_activation(plan, act)
            ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, self.S, b.TSP_WS_FORWARD), dtype=torch.uint8, device="cuda")
            b.tsp_mlp_set_workspace(plan, ws)
            self.Y.fill_(float("nan"))
            b.tsp_mlp_forward(plan, self.X, self.Wg, self.Wu, self.Wd, self.Y, self.S, self.D)
            torch.cuda.synchronize()
            st = b.tsp_mlp_status(plan)
            assert st == b.TSP_OK, f"device status {st} (code {b.tsp_mlp_last_cuda_error(plan)})"
        finally:
            b.tsp_mlp_plan_destroy(plan)
        return self.Y

    def backward(self, act=None):
        """Run tsp_mlp_backward; returns dX (bf16), dWg, dWu, dWd (fp32) torch tensors."""
        import torch

        from paper_2604_26294_b200 import binding as b

        S, H, F, D = self.S, self.H, self.F, self.D
        plan = b.tsp_mlp_plan_ex(H, F, D, **self.options)
        try:
            if act is not None:
                b.tsp_mlp_set_activation(plan, act)
            ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD), dtype=torch.uint8, device="cuda")
            b.tsp_mlp_set_workspace(plan, ws)
            dX = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            dWg = torch.full((D, H, F // D), float("nan"), dtype=torch.float32, device="cuda")
            dWu = torch.full((D, H, F // D), float("nan"), dtype=torch.float32, device="cuda")
            dWd = torch.full((D, F // D, H), float("nan"), dtype=torch.float32, device="cuda")
            b.tsp_mlp_backward(plan, self.X, self.Wg, self.Wu, self.Wd, self.dY, dX, dWg, dWu, dWd, S, D)
            torch.cuda.synchronize()
            st = b.tsp_mlp_status(plan)
            assert st == b.TSP_OK, f"device status {st} (code {b.tsp_mlp_last_cuda_error(plan)})"
        finally:
            b.tsp_mlp_plan_destroy(plan)
        return dX, dWg, dWu, dWd

    def f64(self):
        h = self.host
        out = [inp.bf16_bits_to_f64(h.X), inp.bf16_bits_to_f64(h.Wg), inp.bf16_bits_to_f64(h.Wu),
               inp.bf16_bits_to_f64(h.Wd)]
        if h.dY is not None:
            out.append(inp.bf16_bits_to_f64(h.dY))
        return out
