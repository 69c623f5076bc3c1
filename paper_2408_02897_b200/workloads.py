"""Seeded synthetic inputs with the shapes and distributions of the BERT matmul workloads.

This module only draws numbers and lays them out; it holds none of the probe's arithmetic and
is the one piece of code that both the CUDA path's tests/benchmarks and the CPU oracle's
callers use (they receive the same arrays).

Every generator returns CPU torch tensors.  "bf16 storage" means the fp32 draw rounded to
nearest-even bf16.  An op is a dict:
    name, L (tensor), cl (contracting dim of L), R (tensor), cr (contracting dim of R),
    fmt_l, fmt_r, gran_l, gran_r, ref ("bf16" | "fp32")
with L.R contracted over those dims: out[m, n] = sum_k L[m, k] R[k, n] after orienting.
"""
import numpy as np
import torch


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def normal(rng, shape, std=1.0, dtype=torch.bfloat16):
    x = rng.standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return torch.from_numpy(x).to(dtype)


def student_t(rng, shape, nu, dtype=torch.bfloat16):
    x = rng.standard_t(nu, shape).astype(np.float32)
    return torch.from_numpy(x).to(dtype)


def lognormal_signed(rng, shape, mu, sigma, dtype=torch.bfloat16):
    """Gradient-like values: log-normal magnitudes (the paper finds gradients log-normal), random signs."""
    x = np.exp(rng.normal(mu, sigma, shape)) * rng.choice([-1.0, 1.0], shape)
    return torch.from_numpy(x.astype(np.float32)).to(dtype)


def op(name, L, cl, R, cr, fmt_l, fmt_r, gran_l="tensor", gran_r="tensor", ref="bf16"):
    return dict(name=name, L=L, cl=cl, R=R, cr=cr, fmt_l=fmt_l, fmt_r=fmt_r, gran_l=gran_l,
                gran_r=gran_r, ref=ref)


def config1(seed=0):
    """Single probe: X[128x256], W[256x256] fp32 N(0,1), per-tensor, E4M3, fp32 reference."""
    rng = _rng(seed)
    X = normal(rng, (128, 256), dtype=torch.float32)
    W = normal(rng, (256, 256), dtype=torch.float32)
    return [op("single", X, -1, W, -2, "e4m3", "e4m3", ref="fp32")]


def student_t_example(nu, seed=100, n=512, fmt="int8"):
    """The paper's illustrative example: n x n Student-t matrices, per-vector scaling."""
    rng = _rng(seed)
    L = student_t(rng, (n, n), nu)
    R = student_t(rng, (n, n), nu)
    return [op(f"t{nu}-{fmt}", L, -1, R, -2, fmt, fmt, "channel", "channel")]


def bert_forward_ops(rng, M, H, F, qkv_out, wstd=0.02):
    """Forward matmul operands of one encoder layer: activations N(0,1), weights N(0, wstd^2)."""
    X = normal(rng, (M, H))
    X2 = normal(rng, (M, F))
    return {
        "qkv": (X, normal(rng, (H, qkv_out), wstd)),
        "attn_out": (X, normal(rng, (H, H), wstd)),
        "ffn1": (X, normal(rng, (H, F), wstd)),
        "ffn2": (X2, normal(rng, (F, H), wstd)),
    }


def config2(seed=2, M=4096, H=768, F=3072, formats=("e4m3", "int8")):
    """BERT-base forward matmuls, batch 8 x seq 512; E4M3 and INT8, per-tensor scaling."""
    rng = _rng(seed)
    t = bert_forward_ops(rng, M, H, F, 3 * H)
    ops = []
    for fmt in formats:
        for name, (X, W) in t.items():
            ops.append(op(f"{name}-{fmt}", X, -1, W, -2, fmt, fmt))
    return ops


def config3(seed=3, M=16384, H=1024, F=4096):
    """BERT-large layer, forward + dgrad + wgrad; X, W in E4M3, dY in E5M2 (N(0, 1e-3^2));
    per-channel scales on W, per-tensor on X and dY."""
    rng = _rng(seed)
    t = bert_forward_ops(rng, M, H, F, 3 * H)
    ops = []
    for name, (X, W) in t.items():
        dY = normal(rng, (M, W.shape[1]), 1e-3)
        # fwd  Y = X . W          contract over H: X rows contiguous, W strided
        ops.append(op(f"{name}-fwd", X, -1, W, -2, "e4m3", "e4m3", "tensor", "channel"))
        # dgrad dX = dY . W^T     contract over the output features: both contiguous
        ops.append(op(f"{name}-dgrad", dY, -1, W, -1, "e5m2", "e4m3", "tensor", "channel"))
        # wgrad dW = X^T . dY     contract over the tokens: both strided
        ops.append(op(f"{name}-wgrad", X, -2, dY, -2, "e4m3", "e5m2", "tensor", "tensor"))
    return ops


def config4(seed=4, M=16384, H=1024, F=4096):
    """Outlier stress on the FFN1 shape: Student-t(3) activations, 1% of feature channels x50."""
    rng = _rng(seed)
    x = rng.standard_t(3.0, (M, H)).astype(np.float32)
    cols = rng.choice(H, max(1, H // 100), replace=False)
    x[:, cols] *= np.float32(50.0)
    X = torch.from_numpy(x).to(torch.bfloat16)
    W = normal(rng, (H, F), 0.02)
    ops = []
    for fmt in ("e4m3", "e5m2", "int8"):
        for gran in ("tensor", "channel"):
            ops.append(op(f"ffn1-{fmt}-{gran}", X, -1, W, -2, fmt, fmt, gran, gran))
    return ops


def attention_tensors(rng, batch, S, D):
    """Operands of the score and context products of self-attention, batched over batch =
    examples x heads.  P is the row softmax of Q.K^T / sqrt(D) (input preparation); the upstream
    gradients dS and dO are N(0, 1e-3^2)."""
    Q, K, V = (normal(rng, (batch, S, D)) for _ in range(3))
    P = torch.softmax(torch.matmul(Q.float(), K.float().transpose(1, 2)) / (D ** 0.5), dim=-1).to(torch.bfloat16)
    dS = normal(rng, (batch, S, S), 1e-3)
    dO = normal(rng, (batch, S, D), 1e-3)
    return dict(Q=Q, K=K, V=V, P=P, dS=dS, dO=dO)


def attention_ops(rng, batch, S, D, fmt, tensors=None):
    """Score and context products, forward and backward, for one format of the sweep."""
    t = tensors if tensors is not None else attention_tensors(rng, batch, S, D)
    Q, K, V, P, dS, dO = (t[k] for k in ("Q", "K", "V", "P", "dS", "dO"))
    g = "e5m2" if fmt != "int8" else "int8"      # gradients: E5M2 when the sweep is FP8
    return [
        op(f"qk-fwd-{fmt}", Q, -1, K, -1, fmt, fmt),                  # S = Q . K^T
        op(f"pv-fwd-{fmt}", P, -1, V, -2, fmt, fmt),                  # O = P . V
        op(f"qk-dq-{fmt}", dS, -1, K, -2, g, fmt),                    # dQ = dS . K
        op(f"qk-dk-{fmt}", dS, -2, Q, -2, g, fmt),                    # dK = dS^T . Q
        op(f"pv-dp-{fmt}", dO, -1, V, -1, g, fmt),                    # dP = dO . V^T
        op(f"pv-dv-{fmt}", P, -2, dO, -2, fmt, g),                    # dV = P^T . dO
    ]


# Which tensor category of the paper's Results section each operand of an op belongs to
# (RHS: mostly weights; LHS: activations, inside attention also keys / probabilities; gradient:
# the upstream gradient), and the pass the product belongs to.
_ROLES = {"fwd": ("LHS", "RHS"), "dgrad": ("gradient", "RHS"), "wgrad": ("LHS", "gradient"),
          "qk-fwd": ("LHS", "RHS"), "pv-fwd": ("LHS", "RHS"), "qk-dq": ("gradient", "RHS"),
          "qk-dk": ("gradient", "LHS"), "pv-dp": ("gradient", "RHS"), "pv-dv": ("LHS", "gradient")}


def op_roles(name):
    """(pass, role of L, role of R) of an op of config 3 / 5, from its name."""
    for key, (rl, rr) in _ROLES.items():
        if f"-{key}" in name or name.startswith(key):
            ps = key if key in ("fwd", "dgrad", "wgrad") else ("fwd" if key.endswith("fwd") else "bwd")
            return ps, rl, rr
    return "fwd", "LHS", "RHS"


def config5_layer_tensors(layer, seed=5, M=16384, H=1024, F=4096, heads=16, S=512):
    """The tensors of one layer of the 24-layer sweep (shared by the three formats): projection
    operands with the layer's weight std drawn uniformly in [0.01, 0.05], their upstream
    gradients, and the attention operands."""
    rng = _rng(seed * 1000 + layer)
    wstd = float(rng.uniform(0.01, 0.05))
    proj = bert_forward_ops(rng, M, H, F, 3 * H, wstd)
    grads = {name: normal(rng, (M, W.shape[1]), 1e-3) for name, (X, W) in proj.items()}
    attn = attention_tensors(rng, (M // S) * heads, S, H // heads)
    return dict(layer=layer, wstd=wstd, proj=proj, grads=grads, attn=attn)


def config5_layer(layer, fmt, seed=5, M=16384, H=1024, F=4096, heads=16, S=512, tensors=None):
    """One layer of the 24-layer sweep for one format: 12 projection ops + 6 attention ops,
    per-tensor scales; gradients in E5M2 when the sweep format is an FP8 one."""
    t = tensors if tensors is not None else config5_layer_tensors(layer, seed, M, H, F, heads, S)
    g = "e5m2" if fmt != "int8" else "int8"
    ops = []
    for name, (X, W) in t["proj"].items():
        dY = t["grads"][name]
        ops.append(op(f"L{layer}-{name}-fwd-{fmt}", X, -1, W, -2, fmt, fmt))
        ops.append(op(f"L{layer}-{name}-dgrad-{fmt}", dY, -1, W, -1, g, fmt))
        ops.append(op(f"L{layer}-{name}-wgrad-{fmt}", X, -2, dY, -2, fmt, g))
    for o in attention_ops(None, None, None, None, fmt, tensors=t["attn"]):
        o["name"] = f"L{layer}-" + o["name"]
        ops.append(o)
    return ops


def orient(o):
    """(L as [.., M, K], R as [.., K, N]) float32 numpy views of an op, for CPU-side callers."""
    L = o["L"].float().numpy()
    R = o["R"].float().numpy()
    if o["cl"] == -2:
        L = np.swapaxes(L, -1, -2)
    if o["cr"] == -1:
        R = np.swapaxes(R, -1, -2)
    return L, R


def op_flops(o):
    """(M, N, K, batch) and multiply-add flops (2 M N K batch) of one product."""
    L, R = o["L"], o["R"]
    b = L.shape[0] if L.dim() == 3 else 1
    M = L.shape[-2] if o["cl"] == -1 else L.shape[-1]
    K = L.shape[-1] if o["cl"] == -1 else L.shape[-2]
    N = R.shape[-1] if o["cr"] == -2 else R.shape[-2]
    return (M, N, K, b), 2.0 * M * N * K * b
