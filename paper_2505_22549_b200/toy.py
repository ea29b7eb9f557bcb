"""The paper's toy problem on the CUDA library: noisy Rosenbrock with many workers.

    python -m paper_2505_22549_b200.toy [--steps T] [--lr LR]

f(x1, x2) = (1 - x1)^2 + 100 (x2 - x1^2)^2, M = 256 workers, IID Gaussian gradient noise with
sigma = 1.5, Adam with periods (K_x, K_u, K_v): DES-LOC (192, 192, 692), Local Adam (192, 192, 192)
and FedAvg with local optimizer states (192, never, never).  The paper does not print the
learning rate, betas or step count of its figure, so this is a qualitative demonstration with
settings of our own; it prints the distance of the worker-mean iterate to the optimum (1, 1).
Gradients are evaluated with torch on the GPU at each worker's own iterate; every optimizer
step, averaging included, runs in the library.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as B
from .module import DesLoc


def rosenbrock_grad(x: torch.Tensor) -> torch.Tensor:
    """x: [M, 2] -> gradient [M, 2] of (1-x1)^2 + 100 (x2-x1^2)^2."""
    x1, x2 = x[:, 0], x[:, 1]
    g1 = -2.0 * (1.0 - x1) - 400.0 * x1 * (x2 - x1 * x1)
    g2 = 200.0 * (x2 - x1 * x1)
    return torch.stack([g1, g2], dim=1)


def run(K, steps: int, lr: float, M: int = 256, sigma: float = 1.5, seed: int = 0,
        beta1: float = 0.95, beta2: float = 0.999, device="cuda:0", record=None):
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    X = torch.tensor([-1.0, 1.0], device=dev).repeat(M, 1).contiguous()     # [M, 2]
    U, V = torch.zeros_like(X), torch.zeros_like(X)
    G = torch.zeros_like(X)
    rows = lambda a: [[a[m]] for m in range(M)]
    eng = DesLoc(rows(X), rows(U), rows(V), opt="adam", grad_dtype="f32", beta1=beta1, beta2=beta2,
                 eps=1e-8, clip_rho=0.0, K=K)
    grows = rows(G)
    for t in range(steps):
        G.copy_(rosenbrock_grad(X) + sigma * torch.randn(M, 2, generator=gen, device=dev))
        if record is not None:
            record(t, X, U, V, G)
        eng.step(t, lr, grows)
    torch.cuda.synchronize(dev)
    eng.close()
    return float((X.mean(dim=0) - torch.ones(2, device=dev)).norm())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=6000)
    ap.add_argument("--lr", type=float, default=2e-2)
    a = ap.parse_args()
    for name, K in (("DES-LOC (192,192,692)", (192, 192, 692)), ("Local Adam (192,192,192)", (192, 192, 192)),
                    ("FedAvg, local states (192,-,-)", (192, 0, 0))):
        print(f"{name:34s} distance to optimum after {a.steps} steps: {run(K, a.steps, a.lr):.4f}")


if __name__ == "__main__":
    main()
