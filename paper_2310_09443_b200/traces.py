"""Seeded synthetic training traces (kernel -> tensor CSR) shaped like the paper's workloads.

The paper plans migrations over traces of real models (BERT, ViT, Inceptionv3, ResNet152,
SENet154; Table 1) captured on an A100.  Those traces are not available, so the generators
below build stand-ins with the same structure: a chain of forward kernels, a mirrored chain of
backward kernels, one optimizer kernel per parameter tensor, fp32 byte sizes derived from layer
shapes and kernel durations proportional to FLOPs (Section 4.2 uses profiled kernel times only
to measure how long a tensor stays unused).

This module only *produces inputs*.  It contains none of the method's arithmetic (no vitality,
no pressure, no planning): both the CUDA path and the CPU oracle consume what it returns.
All randomness comes from ``numpy.random.default_rng(seed)`` (PCG64); every float is turned
into an integer once, here.
"""
from __future__ import annotations

import dataclasses
import hashlib
from typing import Callable, List, Optional, Tuple

import numpy as np

GiB = 1 << 30
HOST_BW = 32_000_000_000      # bytes/s, GPU <-> host link (PCIe 4.0 x16 in the paper's SSD-bandwidth sweep)
SSD_BW = 6_400_000_000        # bytes/s, two of the paper's 3.2 GB/s SSDs


@dataclasses.dataclass
class Trace:
    """One training trace in the layout the C-ABI takes (all arrays contiguous, little-endian)."""
    name: str
    kernel_ptr: np.ndarray        # int64[K+1]
    kernel_tensors: np.ndarray    # int32[E]
    tensor_bytes: np.ndarray      # int64[N]
    kernel_ns: np.ndarray         # int64[K]
    tensor_global: np.ndarray     # uint8[N]
    # GPU capacity: either an absolute byte count, or a rational fraction of the unplanned peak
    # pressure (the consumer computes the peak itself and applies floor(peak * num / den)).
    capacity_bytes: Optional[int] = None
    capacity_frac: Optional[Tuple[int, int]] = None
    host_bw: int = HOST_BW
    ssd_bw: int = SSD_BW
    host_capacity_bytes: int = 0  # 0 = unlimited
    kernel_names: Optional[List[str]] = None
    tensor_names: Optional[List[str]] = None

    @property
    def K(self) -> int:
        return int(self.kernel_ns.shape[0])

    @property
    def N(self) -> int:
        return int(self.tensor_bytes.shape[0])

    @property
    def E(self) -> int:
        return int(self.kernel_tensors.shape[0])

    def capacity_from_peak(self, peak_bytes: int) -> int:
        if self.capacity_bytes is not None:
            return int(self.capacity_bytes)
        num, den = self.capacity_frac
        return (int(peak_bytes) * num) // den

    def sha256(self) -> str:
        h = hashlib.sha256()
        for a in (self.kernel_ptr, self.kernel_tensors, self.tensor_bytes, self.kernel_ns, self.tensor_global):
            h.update(np.ascontiguousarray(a).tobytes())
        return h.hexdigest()

    def save(self, path: str) -> str:
        """Write the trace to an .npz file (arrays plus scalars) and return its digest."""
        cap = -1 if self.capacity_bytes is None else int(self.capacity_bytes)
        frac = (0, 0) if self.capacity_frac is None else tuple(int(x) for x in self.capacity_frac)
        np.savez(path, name=np.array(self.name), kernel_ptr=self.kernel_ptr, kernel_tensors=self.kernel_tensors,
                 tensor_bytes=self.tensor_bytes, kernel_ns=self.kernel_ns, tensor_global=self.tensor_global,
                 scalars=np.array([cap, frac[0], frac[1], self.host_bw, self.ssd_bw, self.host_capacity_bytes],
                                  dtype=np.int64))
        return self.sha256()

    @staticmethod
    def load(path: str) -> "Trace":
        """Read back a trace written by :meth:`save`."""
        with np.load(path, allow_pickle=False) as z:
            cap, fnum, fden, host_bw, ssd_bw, host_cap = (int(x) for x in z["scalars"])
            tr = Trace(name=str(z["name"]), kernel_ptr=z["kernel_ptr"].astype(np.int64),
                       kernel_tensors=z["kernel_tensors"].astype(np.int32),
                       tensor_bytes=z["tensor_bytes"].astype(np.int64), kernel_ns=z["kernel_ns"].astype(np.int64),
                       tensor_global=z["tensor_global"].astype(np.uint8),
                       capacity_bytes=None if cap < 0 else cap,
                       capacity_frac=None if fden == 0 else (fnum, fden),
                       host_bw=host_bw, ssd_bw=ssd_bw, host_capacity_bytes=host_cap)
        tr.validate()
        return tr

    def validate(self) -> None:
        assert self.kernel_ptr.dtype == np.int64 and self.kernel_ptr.shape == (self.K + 1,)
        assert self.kernel_tensors.dtype == np.int32
        assert self.tensor_bytes.dtype == np.int64 and self.kernel_ns.dtype == np.int64
        assert self.tensor_global.dtype == np.uint8 and self.tensor_global.shape == (self.N,)
        assert self.kernel_ptr[0] == 0 and self.kernel_ptr[-1] == self.E
        assert np.all(np.diff(self.kernel_ptr) >= 0)
        if self.E:
            assert self.kernel_tensors.min() >= 0 and self.kernel_tensors.max() < self.N
        if self.N:
            assert self.tensor_bytes.min() >= 1 and self.tensor_bytes.max() < (1 << 40)
        if self.K:
            assert self.kernel_ns.min() >= 1 and int(self.kernel_ns.sum()) < (1 << 44)


def from_lists(name: str, kernel_lists, tensor_bytes, kernel_ns, tensor_global=None, **kw) -> Trace:
    """Build a Trace from Python lists (used by tests and by the DNN-shaped generators)."""
    K = len(kernel_lists)
    ptr = np.zeros(K + 1, dtype=np.int64)
    for k, lst in enumerate(kernel_lists):
        ptr[k + 1] = ptr[k] + len(lst)
    flat = [t for lst in kernel_lists for t in lst]
    N = len(tensor_bytes)
    g = np.zeros(N, dtype=np.uint8) if tensor_global is None else np.asarray(tensor_global, dtype=np.uint8)
    return Trace(name=name, kernel_ptr=ptr, kernel_tensors=np.asarray(flat, dtype=np.int32).reshape(-1),
                 tensor_bytes=np.asarray(tensor_bytes, dtype=np.int64).reshape(-1),
                 kernel_ns=np.asarray(kernel_ns, dtype=np.int64).reshape(-1), tensor_global=g, **kw)


# ---------------------------------------------------------------------------------------------
# A tiny tape: forward ops record their kernels and a recipe for the matching backward kernels.
# ---------------------------------------------------------------------------------------------
class _Tape:
    def __init__(self):
        self.t_name: List[str] = []
        self.t_bytes: List[int] = []
        self.t_global: List[int] = []
        self.k_name: List[str] = []
        self.k_list: List[List[int]] = []
        self.k_flops: List[int] = []
        self.backward: List[Callable[[], None]] = []   # run in reverse order
        self.grads = {}                                # tensor id -> list of gradient tensor ids
        self.params: List[Tuple[int, int]] = []        # (param id, grad id) in creation order

    def tensor(self, name: str, nbytes: int, is_global: bool = False) -> int:
        self.t_name.append(name)
        self.t_bytes.append(int(nbytes))
        self.t_global.append(1 if is_global else 0)
        return len(self.t_name) - 1

    def kernel(self, name: str, tensors: List[int], flops: int) -> None:
        self.k_name.append(name)
        self.k_list.append(list(tensors))
        self.k_flops.append(int(flops))

    def add_grad(self, t: int, g: int) -> None:
        self.grads.setdefault(t, []).append(g)

    def grad_of(self, t: int) -> Optional[int]:
        """Gradient of tensor t; several contributions are summed by one n-ary add kernel."""
        gs = self.grads.get(t)
        if not gs:
            return None
        if len(gs) == 1:
            return gs[0]
        nb = self.t_bytes[t]
        s = self.tensor("d(" + self.t_name[t] + ")", nb)
        self.kernel("grad_add", gs + [s], (len(gs) - 1) * (nb // 4))
        self.grads[t] = [s]
        return s

    def run_backward(self) -> None:
        for fn in reversed(self.backward):
            fn()

    def freeze_iteration(self):
        return (self.k_name[:], [l[:] for l in self.k_list], self.k_flops[:])


def _param(tp: _Tape, name: str, nelem: int) -> int:
    return tp.tensor(name, 4 * nelem, is_global=True)


def _param_grad(tp: _Tape, p: int) -> int:
    g = tp.tensor("d" + tp.t_name[p], tp.t_bytes[p])
    tp.params.append((p, g))
    return g


# ---- CNN ops (config 1) ----------------------------------------------------------------------
def _conv(tp: _Tape, x: int, n: int, cin: int, cout: int, k: int, hout: int, name: str, need_dx: bool = True) -> int:
    w = _param(tp, name + ".w", cout * cin * k * k)
    y = tp.tensor(name + ".y", 4 * n * cout * hout * hout)
    flops = 2 * n * cout * hout * hout * cin * k * k
    tp.kernel("conv_fwd:" + name, [x, w, y], flops)

    def bwd():
        dy = tp.grad_of(y)
        dw = _param_grad(tp, w)
        if need_dx:
            dx = tp.tensor("d" + name + ".x", tp.t_bytes[x])
            tp.kernel("conv_bwd_data:" + name, [dy, w, dx], flops)
            tp.add_grad(x, dx)
        tp.kernel("conv_bwd_filter:" + name, [dy, x, dw], flops)
    tp.backward.append(bwd)
    return y


def _bn(tp: _Tape, x: int, c: int, name: str) -> int:
    gamma = _param(tp, name + ".gamma", c)
    beta = _param(tp, name + ".beta", c)
    nb = tp.t_bytes[x]
    y = tp.tensor(name + ".y", nb)
    save = tp.tensor(name + ".save", 8 * c)          # batch mean and inverse std
    tp.kernel("bn_fwd:" + name, [x, gamma, beta, y, save], 4 * (nb // 4))

    def bwd():
        dy = tp.grad_of(y)
        dgamma = _param_grad(tp, gamma)
        dbeta = _param_grad(tp, beta)
        dx = tp.tensor("d" + name + ".x", nb)
        tp.kernel("bn_bwd:" + name, [dy, x, gamma, save, dx, dgamma, dbeta], 8 * (nb // 4))
        tp.add_grad(x, dx)
    tp.backward.append(bwd)
    return y


def _relu(tp: _Tape, x: int, name: str, inplace: bool = False) -> int:
    nb = tp.t_bytes[x]
    if inplace:
        # The paper's instrumented listing calls an in-place ReLU with the same tensor twice.
        tp.kernel("relu_fwd:" + name, [x, x], nb // 4)
        y = x
    else:
        y = tp.tensor(name + ".y", nb)
        tp.kernel("relu_fwd:" + name, [x, y], nb // 4)

    def bwd():
        dy = tp.grad_of(y)
        if inplace:
            tp.kernel("relu_bwd:" + name, [dy, y, dy], nb // 4)
        else:
            dx = tp.tensor("d" + name + ".x", nb)
            tp.kernel("relu_bwd:" + name, [dy, y, dx], nb // 4)
            tp.add_grad(x, dx)
    tp.backward.append(bwd)
    return y


def _add(tp: _Tape, a: int, b: int, name: str) -> int:
    nb = tp.t_bytes[a]
    y = tp.tensor(name + ".y", nb)
    tp.kernel("add_fwd:" + name, [a, b, y], nb // 4)

    def bwd():
        dy = tp.grad_of(y)       # the same gradient flows to both addends: no kernel
        tp.add_grad(a, dy)
        tp.add_grad(b, dy)
    tp.backward.append(bwd)
    return y


def _pool(tp: _Tape, x: int, out_bytes: int, name: str) -> int:
    y = tp.tensor(name + ".y", out_bytes)
    tp.kernel("pool_fwd:" + name, [x, y], tp.t_bytes[x] // 4)

    def bwd():
        dy = tp.grad_of(y)
        dx = tp.tensor("d" + name + ".x", tp.t_bytes[x])
        tp.kernel("pool_bwd:" + name, [dy, x, y, dx], tp.t_bytes[x] // 4)
        tp.add_grad(x, dx)
    tp.backward.append(bwd)
    return y


# ---- Dense / transformer ops (configs 2 and 3) -------------------------------------------------
def _linear(tp: _Tape, x: int, rows: int, din: int, dout: int, name: str, need_dx: bool = True) -> int:
    w = _param(tp, name + ".w", din * dout)
    b = _param(tp, name + ".b", dout)
    y = tp.tensor(name + ".y", 4 * rows * dout)
    flops = 2 * rows * din * dout
    tp.kernel("gemm_fwd:" + name, [x, w, b, y], flops)

    def bwd():
        dy = tp.grad_of(y)
        dw = _param_grad(tp, w)
        db = _param_grad(tp, b)
        if need_dx:
            dx = tp.tensor("d" + name + ".x", tp.t_bytes[x])
            tp.kernel("gemm_bwd_data:" + name, [dy, w, dx], flops)
            tp.add_grad(x, dx)
        tp.kernel("gemm_bwd_weight:" + name, [dy, x, dw, db], flops)
    tp.backward.append(bwd)
    return y


def _bmm(tp: _Tape, a: int, b: int, out_bytes: int, flops: int, name: str) -> int:
    y = tp.tensor(name + ".y", out_bytes)
    tp.kernel("bmm_fwd:" + name, [a, b, y], flops)

    def bwd():
        dy = tp.grad_of(y)
        da = tp.tensor("d" + name + ".a", tp.t_bytes[a])
        db = tp.tensor("d" + name + ".b", tp.t_bytes[b])
        tp.kernel("bmm_bwd_a:" + name, [dy, b, da], flops)
        tp.kernel("bmm_bwd_b:" + name, [dy, a, db], flops)
        tp.add_grad(a, da)
        tp.add_grad(b, db)
    tp.backward.append(bwd)
    return y


def _unary(tp: _Tape, x: int, kind: str, fwd_fpe: int, bwd_fpe: int, name: str, save_input: bool) -> int:
    """Element-wise op (softmax saves its output, GELU saves its input)."""
    nb = tp.t_bytes[x]
    y = tp.tensor(name + ".y", nb)
    tp.kernel(kind + "_fwd:" + name, [x, y], fwd_fpe * (nb // 4))

    def bwd():
        dy = tp.grad_of(y)
        dx = tp.tensor("d" + name + ".x", nb)
        tp.kernel(kind + "_bwd:" + name, [dy, x if save_input else y, dx], bwd_fpe * (nb // 4))
        tp.add_grad(x, dx)
    tp.backward.append(bwd)
    return y


def _layernorm(tp: _Tape, x: int, rows: int, h: int, name: str) -> int:
    gamma = _param(tp, name + ".gamma", h)
    beta = _param(tp, name + ".beta", h)
    nb = tp.t_bytes[x]
    y = tp.tensor(name + ".y", nb)
    stats = tp.tensor(name + ".stats", 8 * rows)
    tp.kernel("ln_fwd:" + name, [x, gamma, beta, y, stats], 8 * (nb // 4))

    def bwd():
        dy = tp.grad_of(y)
        dgamma = _param_grad(tp, gamma)
        dbeta = _param_grad(tp, beta)
        dx = tp.tensor("d" + name + ".x", nb)
        tp.kernel("ln_bwd:" + name, [dy, x, gamma, stats, dx, dgamma, dbeta], 16 * (nb // 4))
        tp.add_grad(x, dx)
    tp.backward.append(bwd)
    return y


def _loss(tp: _Tape, logits: int, name: str = "loss") -> None:
    nb = tp.t_bytes[logits]
    val = tp.tensor(name + ".value", 4)
    tp.kernel("loss_fwd", [logits, val], 8 * (nb // 4))

    def bwd():
        d = tp.tensor("d" + name + ".logits", nb)
        tp.kernel("loss_bwd", [logits, d], 8 * (nb // 4))
        tp.add_grad(logits, d)
    tp.backward.append(bwd)


def _encoder_layer(tp: _Tape, x: int, B: int, S: int, H: int, heads: int, ffn: int, name: str) -> int:
    rows = B * S
    q = _linear(tp, x, rows, H, H, name + ".q")
    k = _linear(tp, x, rows, H, H, name + ".k")
    v = _linear(tp, x, rows, H, H, name + ".v")
    sc_bytes = 4 * B * heads * S * S
    att_flops = 2 * B * S * S * H
    scores = _bmm(tp, q, k, sc_bytes, att_flops, name + ".scores")
    probs = _unary(tp, scores, "softmax", 5, 5, name + ".softmax", save_input=False)
    ctx = _bmm(tp, probs, v, 4 * rows * H, att_flops, name + ".context")
    ao = _linear(tp, ctx, rows, H, H, name + ".out")
    r1 = _add(tp, x, ao, name + ".res1")
    n1 = _layernorm(tp, r1, rows, H, name + ".ln1")
    h1 = _linear(tp, n1, rows, H, ffn, name + ".ffn1")
    g1 = _unary(tp, h1, "gelu", 8, 8, name + ".gelu", save_input=True)
    h2 = _linear(tp, g1, rows, ffn, H, name + ".ffn2")
    r2 = _add(tp, n1, h2, name + ".res2")
    return _layernorm(tp, r2, rows, H, name + ".ln2")


def _optimizer(tp: _Tape, kind: str) -> None:
    """One update kernel per parameter tensor, in parameter-creation order."""
    by_param = {p: g for p, g in tp.params}
    for p in sorted(by_param):
        g = by_param[p]
        nelem = tp.t_bytes[p] // 4
        if kind == "sgd":
            tp.kernel("sgd:" + tp.t_name[p], [g, p], 2 * nelem)
        else:
            m = tp.tensor(tp.t_name[p] + ".adam_m", tp.t_bytes[p], is_global=True)
            v = tp.tensor(tp.t_name[p] + ".adam_v", tp.t_bytes[p], is_global=True)
            tp.kernel("adam:" + tp.t_name[p], [g, p, m, v], 12 * nelem)


def _durations(flops: np.ndarray, rng: np.random.Generator) -> np.ndarray:
    """FLOPs at 50 TFLOP/s in ns (= FLOPs / 50 000), +-20 % uniform jitter, floor of 1 us."""
    u = rng.random(flops.shape[0])
    ns = np.floor(flops.astype(np.float64) / 50_000.0 * (0.8 + 0.4 * u)).astype(np.int64)
    return np.maximum(ns, 1000)


def _finish(tp: _Tape, name: str, rng: np.random.Generator, iterations: int = 1, **kw) -> Trace:
    """Turn a one-iteration tape into a Trace; replicate it if asked (global tensors keep their
    ids across iterations, every other tensor gets a fresh id per iteration)."""
    n1 = len(tp.t_name)
    glob = np.asarray(tp.t_global, dtype=np.uint8)
    inter = np.flatnonzero(glob == 0)
    n_inter = inter.shape[0]
    t_bytes = list(tp.t_bytes)
    t_names = list(tp.t_name)
    t_glob = list(tp.t_global)
    lists = [l[:] for l in tp.k_list]
    names = list(tp.k_name)
    flops = list(tp.k_flops)
    for it in range(1, iterations):
        remap = np.arange(n1, dtype=np.int64)
        remap[inter] = n1 + (it - 1) * n_inter + np.arange(n_inter)
        for i in inter:
            t_bytes.append(tp.t_bytes[i])
            t_names.append(tp.t_name[i] + "@it%d" % it)
            t_glob.append(0)
        for l, nm, f in zip(tp.k_list, tp.k_name, tp.k_flops):
            lists.append([int(remap[t]) for t in l])
            names.append(nm + "@it%d" % it)
            flops.append(f)
    dur = _durations(np.asarray(flops, dtype=np.int64), rng)
    tr = from_lists(name, lists, t_bytes, dur, t_glob, **kw)
    tr.kernel_names = names
    tr.tensor_names = t_names
    tr.validate()
    return tr


# ---------------------------------------------------------------------------------------------
# The five configurations.
# ---------------------------------------------------------------------------------------------
def config0_mlp_chain(seed: int = 0, layers: int = 32) -> Trace:
    """32-layer MLP training step: fwd_1..fwd_L, then for l = L..1: bwd_l, opt_l."""
    rng = np.random.default_rng(seed)
    L = layers
    A = lambda l: l                        # A_0 .. A_L
    dA = lambda l: (L + 1) + l             # dA_0 .. dA_L
    W = lambda l: 2 * (L + 1) + (l - 1)    # W_1 .. W_L
    dW = lambda l: 2 * (L + 1) + L + (l - 1)
    N = 2 * (L + 1) + 2 * L
    lists = []
    for l in range(1, L + 1):
        lists.append([W(l), A(l - 1), A(l)])
    for l in range(L, 0, -1):
        lists.append([A(l - 1), W(l), dA(l), dA(l - 1), dW(l)])
        lists.append([dW(l), W(l)])
    size = np.floor(np.exp2(16.0 + 10.0 * rng.random(N))).astype(np.int64)
    dur = rng.integers(10_000, 2_000_001, size=len(lists)).astype(np.int64)
    glob = np.zeros(N, dtype=np.uint8)
    glob[W(1):W(L) + 1] = 1
    tr = from_lists("c0_mlp_chain", lists, size, dur, glob, capacity_frac=(2, 5))
    tr.validate()
    return tr


def config1_resnet152(seed: int = 1, batch: int = 256, inplace_relu: bool = False) -> Trace:
    """ResNet-152-shaped trace, fp32: stem, bottleneck stages (3, 8, 36, 3), pool, FC, loss; SGD."""
    rng = np.random.default_rng(seed)
    tp = _Tape()
    n = batch
    x = tp.tensor("input", 4 * n * 3 * 224 * 224)
    y = _conv(tp, x, n, 3, 64, 7, 112, "stem.conv", need_dx=False)
    y = _bn(tp, y, 64, "stem.bn")
    y = _relu(tp, y, "stem.relu", inplace_relu)
    y = _pool(tp, y, 4 * n * 64 * 56 * 56, "stem.maxpool")
    cin = 64
    for si, (blocks, mid, hw) in enumerate(zip((3, 8, 36, 3), (64, 128, 256, 512), (56, 28, 14, 7))):
        cout = 4 * mid
        for bi in range(blocks):
            nm = "s%d.b%d" % (si + 1, bi)
            hin = hw * 2 if (bi == 0 and si > 0) else hw
            idt = y
            z = _conv(tp, y, n, cin, mid, 1, hin, nm + ".conv1")
            z = _bn(tp, z, mid, nm + ".bn1")
            z = _relu(tp, z, nm + ".relu1", inplace_relu)
            z = _conv(tp, z, n, mid, mid, 3, hw, nm + ".conv2")       # stride 2 lives here
            z = _bn(tp, z, mid, nm + ".bn2")
            z = _relu(tp, z, nm + ".relu2", inplace_relu)
            z = _conv(tp, z, n, mid, cout, 1, hw, nm + ".conv3")
            z = _bn(tp, z, cout, nm + ".bn3")
            if bi == 0:
                idt = _conv(tp, idt, n, cin, cout, 1, hw, nm + ".down.conv")
                idt = _bn(tp, idt, cout, nm + ".down.bn")
            y = _add(tp, z, idt, nm + ".add")
            y = _relu(tp, y, nm + ".relu3", inplace_relu)
            cin = cout
    y = _pool(tp, y, 4 * n * 2048, "avgpool")
    y = _linear(tp, y, n, 2048, 1000, "fc")
    _loss(tp, y)
    tp.run_backward()
    _optimizer(tp, "sgd")
    return _finish(tp, "c1_resnet152", rng, capacity_bytes=16 * GiB)


def _transformer(name: str, seed: int, layers: int, B: int, S: int, H: int, heads: int, ffn: int,
                 classes: int, capacity: int, iterations: int) -> Trace:
    rng = np.random.default_rng(seed)
    tp = _Tape()
    tok = tp.tensor("tokens", 4 * B * S)
    emb = _param(tp, "embed.table", 30522 * H if name.startswith("c2") else 3 * 14 * 14 * H)
    x = tp.tensor("embed.y", 4 * B * S * H)
    tp.kernel("embed_fwd", [tok, emb, x], B * S * H)

    def emb_bwd():
        dx = tp.grad_of(x)
        demb = _param_grad(tp, emb)
        tp.kernel("embed_bwd", [dx, tok, demb], B * S * H)
    tp.backward.append(emb_bwd)
    for l in range(layers):
        x = _encoder_layer(tp, x, B, S, H, heads, ffn, "l%d" % l)
    y = _linear(tp, x, B * S, H, classes, "head")
    _loss(tp, y)
    tp.run_backward()
    _optimizer(tp, "adam")
    return _finish(tp, name, rng, iterations=iterations, capacity_bytes=capacity)


def config2_bert_large(seed: int = 2) -> Trace:
    """BERT-large-shaped trace: 24 layers, batch 128, seq 512, hidden 1024, 16 heads, FFN 4096, Adam."""
    return _transformer("c2_bert_large", seed, 24, 128, 512, 1024, 16, 4096, 2, 24 * GiB, 1)


def config3_vit_huge(seed: int = 3, iterations: int = 4) -> Trace:
    """ViT-H/14-shaped trace: 32 layers, hidden 1280, MLP 5120, 16 heads, 257 tokens, batch 1024,
    four consecutive training iterations so that parameter tensors idle across iteration boundaries."""
    return _transformer("c3_vit_huge", seed, 32, 1024, 257, 1280, 16, 5120, 1000, 32 * GiB, iterations)


def config4_stress_dag(seed: int = 4, K: int = 1_000_000, N: int = 4_000_000) -> Trace:
    """Scale-stress DAG: tensor i < K is born at kernel i, the rest at uniform kernels; a tensor is
    reused r times with P(r = j) = 0.8 * 0.2^j; reuse gaps are geometric (mean 64 kernels), or
    uniform in [K/100, K/2] for the 5 % long-lived tensors; uses past the last kernel are dropped."""
    rng = np.random.default_rng(seed)
    birth = np.empty(N, dtype=np.int64)
    birth[:K] = np.arange(K)
    birth[K:] = rng.integers(0, K, size=N - K)
    long_lived = rng.random(N) < 0.05
    reuse = rng.geometric(0.8, size=N) - 1
    ev_t = [np.arange(N, dtype=np.int64)]
    ev_k = [birth.copy()]
    cur = birth.copy()
    alive = np.arange(N, dtype=np.int64)
    lo, hi = max(1, K // 100), max(2, K // 2)
    j = 0
    while alive.size:
        alive = alive[reuse[alive] > j]
        if not alive.size:
            break
        gap = rng.geometric(1.0 / 64.0, size=alive.size).astype(np.int64)
        lg = rng.integers(lo, hi + 1, size=alive.size)
        gap = np.where(long_lived[alive], lg, gap)
        nxt = cur[alive] + gap
        keep = nxt <= K - 1
        alive = alive[keep]
        cur[alive] = nxt[keep]
        ev_t.append(alive.copy())
        ev_k.append(cur[alive].copy())
        j += 1
    t = np.concatenate(ev_t)
    k = np.concatenate(ev_k)
    order = np.lexsort((t, k))
    t, k = t[order], k[order]
    ptr = np.zeros(K + 1, dtype=np.int64)
    np.cumsum(np.bincount(k, minlength=K), out=ptr[1:])
    size = np.floor(rng.lognormal(np.log(4 * 1024 * 1024), 1.5, size=N))
    size = np.clip(size, 4096, 2 * GiB).astype(np.int64)
    dur = np.maximum(1, np.floor(rng.lognormal(np.log(100_000.0), 1.0, size=K))).astype(np.int64)
    tr = Trace(name="c4_stress_dag" if (K, N) == (1_000_000, 4_000_000) else "c4_stress_dag_K%d_N%d" % (K, N),
               kernel_ptr=ptr, kernel_tensors=t.astype(np.int32), tensor_bytes=size, kernel_ns=dur,
               tensor_global=np.zeros(N, dtype=np.uint8), capacity_frac=(3, 10))
    tr.validate()
    return tr


def random_toy(rng: np.random.Generator, K: int, N: int, max_deg: int = 4, dup_prob: float = 0.15,
               global_prob: float = 0.25, max_bytes: int = 64, max_ns: int = 40) -> Trace:
    """Small random trace with empty kernels, repeated tensor ids inside a kernel and unused tensors."""
    lists = []
    for _ in range(K):
        deg = int(rng.integers(0, max_deg + 1))
        lst = [int(v) for v in rng.integers(0, N, size=deg)] if N else []
        if lst and rng.random() < dup_prob:
            lst.append(lst[int(rng.integers(0, len(lst)))])
        lists.append(lst)
    size = rng.integers(1, max_bytes + 1, size=N)
    dur = rng.integers(1, max_ns + 1, size=K)
    glob = (rng.random(N) < global_prob).astype(np.uint8)
    return from_lists("toy", lists, size, dur, glob, capacity_frac=(1, 2),
                      host_bw=int(rng.integers(1, 9)) * 1_000_000_000, ssd_bw=int(rng.integers(1, 5)) * 500_000_000)


CONFIGS = {
    0: config0_mlp_chain,
    1: config1_resnet152,
    2: config2_bert_large,
    3: config3_vit_huge,
    4: config4_stress_dag,
}


def make_config(index: int, **kw) -> Trace:
    return CONFIGS[index](**kw)
