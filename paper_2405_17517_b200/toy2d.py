"""The paper's 2-D illustration (Appendix, "2D optimization example") on top of the library.

Two models of two parameters each descend a simplified Ackley function with two local minima,
(3, 8) and (8, 3), and a global one at (10, 10), from (0, 5) and (5, 0): exact gradient plus
Gaussian noise, learning rate 0.1, 1000 steps.  Trained apart they settle in different local
minima; with WASH (p = 0.01 for both coordinates) they exchange coordinates now and then, and
with PAPA they are pulled toward their mean (alpha = 0.99).  The paper gives no noise scale, so
the outcome is qualitative; `noise = 0` makes a run depend on the shuffle's draws alone.

The gradient step runs on the host in binary32; the population operators run in the library
through `wash_step_host` (`LibraryOps`), on a stack of N = 2 rows of one 2-element tensor.

    python -m paper_2405_17517_b200.toy2d [noise]
"""
from __future__ import annotations

import sys

import numpy as np

START = ((0.0, 5.0), (5.0, 0.0))
MINIMA = ((10.0, 10.0, 10.0, 0.1), (5.0, 8.0, 3.0, 0.3), (5.0, 3.0, 8.0, 0.3))   # weight, x_m, y_m, lambda
ROW = 8   # a row holds the 2 parameters and 6 elements of padding


def loss(x: float, y: float) -> float:
    """f(x, y) = -10 g(.,10,10,0.1) - 5 g(.,8,3,0.3) - 5 g(.,3,8,0.3),  g = exp(-lambda sqrt(((x-xm)^2+(y-ym)^2)/2))"""
    return -sum(w * np.exp(-lam * np.sqrt(0.5 * ((x - xm) ** 2 + (y - ym) ** 2))) for w, xm, ym, lam in MINIMA)


def gradient(x: float, y: float):
    gx = gy = 0.0
    for w, xm, ym, lam in MINIMA:
        r = np.sqrt(0.5 * ((x - xm) ** 2 + (y - ym) ** 2))
        if r > 0.0:
            k = w * lam * np.exp(-lam * r) * 0.5 / r
            gx += k * (x - xm)
            gy += k * (y - ym)
    return gx, gy


class LibraryOps:
    """Shuffle and EMA of the 2 x ROW host stack through the C ABI (one GPU)."""

    def __init__(self, device: int = 0):
        import torch
        from . import binding as B
        self.B, self.torch = B, torch
        self.pop = B.Population(2, [2], B.WASH_LAYOUT_NP, device)
        assert self.pop.padded_P == ROW
        self.dev = torch.zeros(2 * ROW, dtype=torch.float32, device="cuda:%d" % device)
        self.pop.bind(B.WASH_STACK_PARAMS, self.dev)
        self.host = torch.zeros(2 * ROW, dtype=torch.float32).pin_memory()

    def _run(self, stack: np.ndarray, ops: int, step: int, p: float, seed: int, alpha: float) -> None:
        self.host.numpy()[:] = stack.reshape(-1)
        self.B.wash_step_host(self.pop.ctx, ops, self.host, None, None, step, p, None, seed, alpha)
        stack.reshape(-1)[:] = self.host.numpy()

    def shuffle(self, stack, step, p, seed):
        self._run(stack, self.B.WASH_OP_SHUFFLE, step, p, seed, 0.5)

    def ema(self, stack, alpha):
        self._run(stack, self.B.WASH_OP_EMA, 0, 0.0, 0, alpha)

    def close(self):
        self.pop.close()


def run(method: str, ops, noise: float = 0.0, seed: int = 0, steps: int = 1000, lr: float = 0.1, p: float = 0.01,
        alpha: float = 0.99, ema_every: int = 10, trace=None) -> np.ndarray:
    """method: "baseline" (no communication), "wash" (shuffle after every step) or "papa" (EMA every
    `ema_every` steps).  Returns the two models' final (x, y); `trace` (a list) receives the stack's
    bit patterns after every step."""
    rng = np.random.default_rng(seed)
    stack = np.zeros((2, ROW), dtype=np.float32)
    stack[0, :2], stack[1, :2] = START
    for t in range(steps):
        for n in range(2):
            gx, gy = gradient(float(stack[n, 0]), float(stack[n, 1]))
            nz = rng.standard_normal(2) * noise
            stack[n, 0] = np.float32(stack[n, 0] - np.float32(lr * (gx + nz[0])))
            stack[n, 1] = np.float32(stack[n, 1] - np.float32(lr * (gy + nz[1])))
        if method == "wash":
            ops.shuffle(stack, t, p, seed)
        elif method == "papa" and t % ema_every == ema_every - 1:
            ops.ema(stack, alpha)
        if trace is not None:
            trace.append(stack.view(np.uint32).copy())
    return stack[:, :2].copy()


if __name__ == "__main__":
    noise_arg = float(sys.argv[1]) if len(sys.argv) > 1 else 0.0
    lib = LibraryOps()
    for name in ("baseline", "papa", "wash"):
        end = run(name, lib, noise=noise_arg)
        print("%-8s model 0 -> (%.2f, %.2f) f = %.2f   model 1 -> (%.2f, %.2f) f = %.2f" % (
            name, end[0, 0], end[0, 1], loss(*end[0]), end[1, 0], end[1, 1], loss(*end[1])))
    lib.close()
