"""Seeded synthetic layer-pruning workloads.

This module only draws random inputs (calibration activations X, dense weight W
and the pruning budget); it holds none of the pruning method's arithmetic.  Both
the CPU oracle's tests and the CUDA path's tests/benchmarks take their inputs
from here so that the two sides see identical arrays.

Every generator is a pure function of its arguments and `seed`.  Large
activation matrices are produced chunk by chunk (`rows` = a slice of tokens):
chunk `c` of a workload is drawn from a generator seeded with
`seed * 1_000_003 + 7919 * (c + 1)`, so a chunk can be regenerated at any time
without holding the whole matrix.

The five named configurations mirror the layer shapes the paper prunes
(Section 2 "Problem Formulation": dense layers, convolutional input channels,
attention heads and FC2 neurons of OPT-style blocks; Section 4 calibration of
128 segments x 2048 tokens).  The paper's models and datasets are not available
here, so these inputs stand in for them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Iterator, Optional

import torch

CHUNK_ROWS = 16384


@dataclass
class Workload:
    """Description of one synthetic layer; activations come from `x_chunks()`."""

    name: str
    kind: str                 # "dense_mix" | "fc2_relu" | "attn_heads" | "conv_unfold" | "conv1x1"
    n: int                    # calibration rows (tokens / patches)
    d1: int                   # rows of W (inputs)
    m: int                    # columns of W (outputs)
    g: int                    # rows per group
    k: int                    # groups kept
    max_swaps: int
    x_dtype: torch.dtype
    seed: int = 0
    damp: float = 0.0
    eps_acc: float = 1e-5               # a swap is accepted iff it lowers obj by more than eps_acc * obj
    score_mode: str = "independent"     # or "pair_exact"
    w_std: float = 0.02
    chunk_rows: int = CHUNK_ROWS
    params: dict = field(default_factory=dict)

    @property
    def ngroups(self) -> int:
        return self.d1 // self.g

    @property
    def n_chunks(self) -> int:
        return (self.n + self.chunk_rows - 1) // self.chunk_rows

    # ------------------------------------------------------------------ W
    def weight(self, device: str = "cpu") -> torch.Tensor:
        gen = torch.Generator(device="cpu").manual_seed(self.seed * 1_000_003 + 11)
        W = torch.randn(self.d1, self.m, generator=gen, dtype=torch.float32) * self.w_std
        return W.to(device)

    # ------------------------------------------------------------------ X
    def _shared(self, device: str):
        """Per-workload random structure shared by every chunk."""
        if hasattr(self, "_shared_cache") and self._shared_cache[0] == device:
            return self._shared_cache[1]
        gen = torch.Generator(device="cpu").manual_seed(self.seed * 1_000_003 + 23)
        out = {}
        if self.kind in ("dense_mix", "conv1x1"):
            E = torch.randn(self.d1, self.d1, generator=gen, dtype=torch.float32) / math.sqrt(self.d1)
            out["A"] = (torch.eye(self.d1) + self.params.get("mix", 0.3) * E).to(device)
        elif self.kind == "fc2_relu":
            r = self.params.get("rank", 64)
            out["U"] = torch.randn(self.d1, r, generator=gen, dtype=torch.float32).to(device)
            out["Vm"] = torch.randn(r, self.d1, generator=gen, dtype=torch.float32).to(device)
        if self.params.get("outlier_frac", 0.0) > 0:
            n_out = max(1, int(round(self.params["outlier_frac"] * self.d1)))
            idx = torch.randperm(self.d1, generator=gen)[:n_out].sort().values
            scale = torch.ones(self.d1, dtype=torch.float32)
            scale[idx] = self.params["outlier_scale"]
            out["scale"] = scale.to(device)
            out["outlier_idx"] = idx
        self._shared_cache = (device, out)
        return out

    def x_chunk(self, c: int, device: str = "cpu") -> torch.Tensor:
        """Rows [c*chunk_rows, min(n, (c+1)*chunk_rows)) of X in `x_dtype`.

        With device="cuda" the normal draws come from the CUDA generator (same
        distribution, different stream than the CPU one); tests that compare
        against the oracle use the default CPU stream.
        """
        r0 = c * self.chunk_rows
        rows = min(self.n, r0 + self.chunk_rows) - r0
        if rows <= 0:
            raise IndexError(c)
        sh = self._shared(device)
        gdev = "cuda" if str(device).startswith("cuda") else "cpu"
        gen = torch.Generator(device=gdev).manual_seed(self.seed * 1_000_003 + 7919 * (c + 1))

        def randn(*shape):
            return torch.randn(*shape, generator=gen, dtype=torch.float32, device=device)

        if self.kind == "dense_mix":
            X = randn(rows, self.d1) @ sh["A"]
        elif self.kind == "fc2_relu":
            Z = randn(rows, self.d1)
            r = sh["U"].shape[1]
            rho = self.params.get("rho", 1.0)
            pre = Z + (rho / math.sqrt(r * self.d1)) * ((Z @ sh["U"]) @ sh["Vm"])
            X = torch.relu_(pre)
        elif self.kind == "attn_heads":
            dh = self.g
            corr = self.params.get("corr", 0.5)
            s = randn(rows, self.d1 // dh, 1)
            z = randn(rows, self.d1 // dh, dh)
            X = (math.sqrt(corr) * s + math.sqrt(1.0 - corr) * z).reshape(rows, self.d1)
        elif self.kind == "conv_unfold":
            # `rows` patches = images * fh * fw; a chunk always holds whole images
            cin, kh, kw = self.d1 // self.g, self.params["kh"], self.params["kw"]
            fh, fw = self.params["fh"], self.params["fw"]
            imgs = rows // (fh * fw)
            F = torch.relu_(randn(imgs, cin, fh, fw))
            cols = torch.nn.functional.unfold(F, (kh, kw), padding=self.params["pad"], stride=1)
            # cols: imgs x (cin*kh*kw) x (fh*fw), row index of the middle axis = c*kh*kw + i*kw + j
            X = cols.transpose(1, 2).reshape(imgs * fh * fw, self.d1)
        elif self.kind == "conv1x1":
            # pointwise convolution: every pixel of the cin-channel feature map is one row; channels are mixed by a
            # fixed random matrix before the ReLU so that they are correlated, as the outputs of a depthwise stage are
            cin, fh, fw = self.d1, self.params["fh"], self.params["fw"]
            imgs = rows // (fh * fw)
            F = torch.relu_(randn(imgs * fh * fw, cin) @ sh["A"])
            X = F
        else:
            raise ValueError(self.kind)
        if "scale" in sh:
            X = X * sh["scale"]
        return X.to(self.x_dtype).contiguous()

    # ------------------------------------------------------------------ sequential layer-wise setting
    def x_pruned_chunk(self, c: int, device: str = "cpu", noise: float = 0.1) -> torch.Tensor:
        """Input block as the already-pruned upstream model would produce it: the dense block plus a seeded
        perturbation of relative size `noise` (same dtype and sign structure)."""
        X = self.x_chunk(c, device).float()
        gdev = "cuda" if str(device).startswith("cuda") else "cpu"
        gen = torch.Generator(device=gdev).manual_seed(self.seed * 1_000_003 + 104729 * (c + 1))
        E = torch.randn(X.shape, generator=gen, dtype=torch.float32, device=device)
        Xp = X + noise * X.abs().mean() * E
        if self.kind in ("fc2_relu", "conv_unfold"):
            Xp = torch.relu_(Xp)
        return Xp.to(self.x_dtype).contiguous()

    def dense_output_chunk(self, c: int, device: str = "cpu", dtype: torch.dtype = torch.float32) -> torch.Tensor:
        """Y block = dense-model input block times the dense weight (the layer's target output)."""
        Y = self.x_chunk(c, device).double() @ self.weight(device).double()
        return Y.to(dtype).contiguous()

    def x_chunks(self, device: str = "cpu") -> Iterator[torch.Tensor]:
        for c in range(self.n_chunks):
            yield self.x_chunk(c, device)

    def x_full(self, device: str = "cpu") -> torch.Tensor:
        return torch.cat(list(self.x_chunks(device)), dim=0)


# ---------------------------------------------------------------------- named configurations
def config(name: str, seed: int = 0, **over) -> Workload:
    """The named layer shapes (c1..c5 of the headline set, c6 a pointwise convolution) and scaled-down relatives.

    `over` replaces any Workload field (e.g. n=4096, d1=1024) to get a smaller
    problem with the same value structure.
    """
    name = name.lower()
    if name == "c1":      # single dense layer, correlated columns
        wl = Workload("c1", "dense_mix", n=256, d1=64, m=64, g=1, k=32, max_swaps=50,
                      x_dtype=torch.float32, w_std=1.0 / 8.0, params={"mix": 0.3})
    elif name == "c2":    # OPT-1.3B-shaped FC2 neurons
        wl = Workload("c2", "fc2_relu", n=262144, d1=8192, m=2048, g=1, k=4096, max_swaps=2000,
                      x_dtype=torch.bfloat16, damp=1e-2, eps_acc=1e-7, params={"rank": 64, "rho": 1.0})
    elif name == "c3":    # OPT-2.7B-shaped attention heads
        wl = Workload("c3", "attn_heads", n=262144, d1=2560, m=2560, g=80, k=16, max_swaps=200,
                      x_dtype=torch.bfloat16, damp=1e-2, eps_acc=1e-7, score_mode="pair_exact",
                      params={"corr": 0.5, "outlier_frac": 0.01, "outlier_scale": 20.0})
    elif name == "c4":    # ResNet50-shaped 3x3 conv input channels
        wl = Workload("c4", "conv_unfold", n=6272, d1=4608, m=512, g=9, k=256, max_swaps=500,
                      x_dtype=torch.float32, w_std=math.sqrt(2.0 / 4608.0),
                      chunk_rows=6272, params={"kh": 3, "kw": 3, "fh": 7, "fw": 7, "pad": 1})
    elif name == "c5":    # OPT-30B-shaped FC2 neurons with outlier channels
        wl = Workload("c5", "fc2_relu", n=262144, d1=28672, m=7168, g=1, k=8602, max_swaps=5000,
                      x_dtype=torch.bfloat16, damp=1e-2, eps_acc=1e-7,
                      params={"rank": 64, "rho": 1.0, "outlier_frac": 0.005, "outlier_scale": 30.0})
    elif name == "c6":    # MobileNetV1-shaped pointwise (1x1) convolution: input channels, 500 images of 7 x 7
        wl = Workload("c6", "conv1x1", n=500 * 49, d1=1024, m=1024, g=1, k=512, max_swaps=500,
                      x_dtype=torch.float32, w_std=math.sqrt(2.0 / 1024.0), chunk_rows=100 * 49,
                      params={"mix": 0.5, "fh": 7, "fw": 7})
    else:
        raise ValueError(name)
    wl.seed = seed
    for key, val in over.items():
        if key == "params":
            wl.params.update(val)
        else:
            setattr(wl, key, val)
    if wl.kind == "conv1x1":
        hw = wl.params["fh"] * wl.params["fw"]
        assert wl.n % hw == 0 and wl.chunk_rows % hw == 0, "conv chunks must hold whole images"
    if wl.kind == "conv_unfold":
        hw = wl.params["fh"] * wl.params["fw"]
        assert wl.n % hw == 0 and wl.chunk_rows % hw == 0, "conv chunks must hold whole images"
        wl.w_std = over.get("w_std", math.sqrt(2.0 / wl.d1))
    assert wl.d1 % wl.g == 0 and 1 <= wl.k <= wl.ngroups
    return wl


def tiny(p: int = 12, m: int = 5, g: int = 1, k: int = 6, n: int = 40, seed: int = 0,
         mix: float = 0.6) -> Workload:
    """Small dense problem for exhaustive checks (all supports can be enumerated)."""
    return Workload(f"tiny_p{p}_g{g}", "dense_mix", n=n, d1=p * g, m=m, g=g, k=k, max_swaps=50,
                    x_dtype=torch.float32, seed=seed, w_std=1.0, chunk_rows=n, params={"mix": mix})
