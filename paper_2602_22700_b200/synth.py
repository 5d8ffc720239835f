"""Seeded synthetic inputs for the sumcheck matmul prover (shared by tests, bench and oracle
checks; holds none of the prover's arithmetic).

Everything is integer-only and built from one counter-based generator, so the same call gives
identical bits on the CPU and on a CUDA device:

    mix64   = the SplitMix64 output mixer
    key     = mix64(mix64(seed + G) + G*(tid+1))
    u(idx)  = mix64(key + G*(idx+1)),  G = 0x9E3779B97F4A7C15,  all mod 2^64

``tid`` names a tensor: (group << 8) | role, group = layer or expert index, role 0 = activation,
1 = weight (or W_up), 2 = W_down, 3 = router, 4.. = further activations.

Value recipes
  uniform int8 in [-127,127]:  ((u >> 32) * 255 >> 32) - 127
  approx-Gaussian int8:        S = sum of the 8 bytes of u (mean 1020, std ~209);
                               clamp(((S-1020)*q + 32768) >> 16, -127, 127) with q = 6271 for
                               sigma 20 and q = 2508 for sigma 8 (support ~4.9 sigma, so the clip
                               never binds)

The layer shapes stand in for the transformer layers of the models the paper audits
(4096-wide residual stream, 14336 FFN, 6144 fused QKV, 8 experts with top-2 routing); no trained
weights or dataset prompts are involved.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import torch

_M64 = (1 << 64) - 1
_G = 0x9E3779B97F4A7C15
Q_SIGMA20 = 6271
Q_SIGMA8 = 2508

ROLE_ACT, ROLE_W, ROLE_W_DOWN, ROLE_ROUTER, ROLE_ACT2, ROLE_ACT3, ROLE_ACT4 = 0, 1, 2, 3, 4, 5, 6


def _s64(x: int) -> int:
    """Python int (mod 2^64) -> the signed 64-bit value with the same bit pattern."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix64_py(z: int) -> int:
    z &= _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 bit patterns."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(0xBF58476D1CE4E5B9)
    z = (z ^ _lsr(z, 27)) * _s64(0x94D049BB133111EB)
    return z ^ _lsr(z, 31)


def stream_key(seed: int, tid: int) -> int:
    return _mix64_py(_mix64_py(seed + _G) + _G * (tid + 1))


def stream_u64(seed: int, tid: int, idx: torch.Tensor) -> torch.Tensor:
    """u(idx) as int64 bit patterns; idx is an int64 tensor of counters."""
    key = stream_key(seed, tid)
    return _mix64((idx + 1) * _s64(_G) + _s64(key))


def _fill(seed: int, tid: int, rows: int, cols: int, device, fn, chunk_elems: int = 1 << 24,
          dtype=torch.int8):
    out = torch.empty((rows, cols), dtype=dtype, device=device)
    flat = out.view(-1)
    total = rows * cols
    for start in range(0, total, chunk_elems):
        stop = min(total, start + chunk_elems)
        idx = torch.arange(start, stop, dtype=torch.int64, device=device)
        flat[start:stop] = fn(stream_u64(seed, tid, idx)).to(dtype)
    return out


def uniform_i8(seed: int, tid: int, rows: int, cols: int, device="cpu") -> torch.Tensor:
    def fn(u):
        return ((_lsr(u, 32) * 255) >> 32) - 127

    return _fill(seed, tid, rows, cols, device, fn)


def byte_sum(u: torch.Tensor) -> torch.Tensor:
    s = u & 0xFF
    for b in range(1, 8):
        s = s + (_lsr(u, 8 * b) & 0xFF)
    return s


def gauss_i8(seed: int, tid: int, rows: int, cols: int, q: int, device="cpu") -> torch.Tensor:
    def fn(u):
        return torch.clamp(((byte_sum(u) - 1020) * q + 32768) >> 16, -127, 127)

    return _fill(seed, tid, rows, cols, device, fn)


def exact_matmul_i32(A: torch.Tensor, B: torch.Tensor, row_chunk: int = 4096) -> torch.Tensor:
    """Exact int8 x int8 -> int32 product used only to manufacture the claimed matrix C.

    On a CUDA device it uses the library integer GEMM where its shape rules allow, else fp32
    products over chunks of 1024 along k (every partial sum is an integer below 2^24, so fp32
    accumulation in any order is exact; TF32 is switched off for the call)."""
    m, k = A.shape
    k2, n = B.shape
    assert k == k2
    if A.device.type == "cpu":
        return (A.to(torch.int32) @ B.to(torch.int32)).contiguous()
    C = torch.empty((m, n), dtype=torch.int32, device=A.device)
    use_int_mm = hasattr(torch, "_int_mm") and k % 8 == 0 and n % 8 == 0
    for r0 in range(0, m, row_chunk):
        r1 = min(m, r0 + row_chunk)
        Ab = A[r0:r1]
        done = False
        if use_int_mm and (r1 - r0) > 16:
            try:
                C[r0:r1] = torch._int_mm(Ab.contiguous(), B)
                done = True
            except RuntimeError:
                use_int_mm = False
        if not done:
            tf32 = torch.backends.cuda.matmul.allow_tf32
            torch.backends.cuda.matmul.allow_tf32 = False
            try:
                acc = torch.zeros((r1 - r0, n), dtype=torch.int32, device=A.device)
                for c0 in range(0, k, 1024):
                    c1 = min(k, c0 + 1024)
                    part = Ab[:, c0:c1].to(torch.float32) @ B[c0:c1].to(torch.float32)
                    acc += part.to(torch.int32)
                C[r0:r1] = acc
            finally:
                torch.backends.cuda.matmul.allow_tf32 = tf32
    return C


def requantize_i8(C: torch.Tensor) -> torch.Tensor:
    """int32 FFN hidden -> int8 input of the down projection: clamp((C + 256) >> 9, -127, 127), with the
    sum taken without 32-bit wrap-around: (C >> 9) + (((C & 511) + 256) >> 9)."""
    return torch.clamp((C >> 9) + (((C & 511) + 256) >> 9), -127, 127).to(torch.int8)


# ---------------------------------------------------------------------------- workloads


@dataclass
class Problem:
    """One claimed product C = A*B with the proof id its challenges are drawn under."""
    name: str
    A: torch.Tensor          # m x k int8
    B: torch.Tensor          # k x n int8
    C: torch.Tensor          # m x n int32 (the CLAIMED product; exact unless tampered with)
    proof_id: int

    @property
    def mkn(self):
        return self.A.shape[0], self.A.shape[1], self.B.shape[1]


def tid(group: int, role: int) -> int:
    return (group << 8) | role


def single_small(seed: int = 1, m: int = 64, k: int = 64, n: int = 64, device="cpu") -> List[Problem]:
    """Uniform int8 operands, one proof (the 64x64x64 case by default)."""
    A = uniform_i8(seed, tid(0, ROLE_ACT), m, k, device)
    B = uniform_i8(seed, tid(0, ROLE_W), k, n, device)
    return [Problem("small", A, B, exact_matmul_i32(A, B), 0)]


def qkv_projection(seed: int = 1, tokens: int = 512, d_model: int = 4096, d_out: int = 4096,
                   device="cpu") -> List[Problem]:
    """Dense-layer projection: Gaussian activations (sigma 20) times Gaussian weights (sigma 8)."""
    A = gauss_i8(seed, tid(0, ROLE_ACT), tokens, d_model, Q_SIGMA20, device)
    B = gauss_i8(seed, tid(0, ROLE_W), d_model, d_out, Q_SIGMA8, device)
    return [Problem("qkv", A, B, exact_matmul_i32(A, B), 0)]


def ffn_pair(seed: int = 1, tokens: int = 2048, d_model: int = 4096, d_ff: int = 14336,
             device="cpu") -> List[Problem]:
    """FFN up projection, int8 requantisation of the hidden, then the down projection.  The
    requantisation only manufactures the next int8 input; it is not part of what is proved."""
    A = gauss_i8(seed, tid(0, ROLE_ACT), tokens, d_model, Q_SIGMA20, device)
    Wu = gauss_i8(seed, tid(0, ROLE_W), d_model, d_ff, Q_SIGMA8, device)
    Cu = exact_matmul_i32(A, Wu)
    H = requantize_i8(Cu)
    Wd = gauss_i8(seed, tid(0, ROLE_W_DOWN), d_ff, d_model, Q_SIGMA8, device)
    return [Problem("ffn_up", A, Wu, Cu, 0), Problem("ffn_down", H, Wd, exact_matmul_i32(H, Wd), 1)]


def moe_routing(seed: int, tokens: int, experts: int, top: int = 2, device="cpu") -> List[torch.Tensor]:
    """Token indices (ascending) routed to each expert.  Logit of (token t, expert e) is the
    centred byte sum of u(experts*t + e) under the router tensor id; the ``top`` largest win,
    ties going to the lower expert index."""
    idx = torch.arange(tokens * experts, dtype=torch.int64, device=device)
    logits = (byte_sum(stream_u64(seed, tid(0, ROLE_ROUTER), idx)) - 1020).view(tokens, experts)
    # stable ordering with ties to the lower index: sort by (-logit, index)
    keyed = (-logits) * experts + torch.arange(experts, device=device, dtype=torch.int64)
    order = torch.argsort(keyed, dim=1)[:, :top]
    chosen = torch.zeros((tokens, experts), dtype=torch.bool, device=device)
    chosen.scatter_(1, order, True)
    return [torch.nonzero(chosen[:, e]).view(-1) for e in range(experts)]


def moe_experts(seed: int = 1, tokens: int = 4096, d_model: int = 4096, d_ff: int = 14336,
                experts: int = 8, top: int = 2, device="cpu") -> List[Problem]:
    """One ragged GEMM per expert: the routed rows of one activation matrix times W_e."""
    X = gauss_i8(seed, tid(0, ROLE_ACT), tokens, d_model, Q_SIGMA20, device)
    routed = moe_routing(seed, tokens, experts, top, device)
    out = []
    for e in range(experts):
        if routed[e].numel() == 0:
            continue
        Ae = X.index_select(0, routed[e]).contiguous()
        We = gauss_i8(seed, tid(e, ROLE_W), d_model, d_ff, Q_SIGMA8, device)
        out.append(Problem(f"expert{e}", Ae, We, exact_matmul_i32(Ae, We), e))
    return out


# roles of the four matmuls of one decoder layer: (activation role, weight role)
_BLOCK_ROLES = (("qkv", 0, 1), ("o", 4, 5), ("up", 6, 7), ("down", 8, 2))


def decoder_block(seed: int = 1, layers: int = 32, tokens: int = 8192, d_model: int = 4096,
                  d_qkv: int = 6144, d_ff: int = 14336, device="cpu") -> List[Problem]:
    """Four proved matmuls per layer (QKV, O, FFN up, FFN down) with independent synthetic
    activations; proof_id = 4*layer + {0,1,2,3}."""
    shapes = {"qkv": (d_model, d_qkv), "o": (d_model, d_model), "up": (d_model, d_ff),
              "down": (d_ff, d_model)}
    out = []
    for layer in range(layers):
        for slot, (name, ra, rw) in enumerate(_BLOCK_ROLES):
            k, n = shapes[name]
            A = gauss_i8(seed, tid(layer, ra), tokens, k, Q_SIGMA20, device)
            W = gauss_i8(seed, tid(layer, rw), k, n, Q_SIGMA8, device)
            out.append(Problem(f"L{layer}.{name}", A, W, exact_matmul_i32(A, W), 4 * layer + slot))
    return out


ROLE_Q, ROLE_KT, ROLE_P, ROLE_V = 9, 10, 11, 12


def attention_block(seed: int = 1, layers: int = 8, tokens: int = 2048, heads: int = 32, head_dim: int = 128,
                    device="cpu") -> List[Problem]:
    """The two matrix products inside attention, per layer and head: scores S = Q K^T (k = head_dim,
    C is tokens x tokens) and outputs O = P V (k = tokens).  K is generated already transposed
    (head_dim x tokens); P is an independent int8 stand-in for the requantised probabilities (the
    softmax between the two products is not part of what is proved).  proof_id counts the products."""
    out = []
    for layer in range(layers):
        for h in range(heads):
            g = layer * heads + h
            Q = gauss_i8(seed, tid(g, ROLE_Q), tokens, head_dim, Q_SIGMA20, device)
            Kt = gauss_i8(seed, tid(g, ROLE_KT), head_dim, tokens, Q_SIGMA20, device)
            out.append(Problem(f"L{layer}.h{h}.qk", Q, Kt, exact_matmul_i32(Q, Kt), 2 * g))
            P = gauss_i8(seed, tid(g, ROLE_P), tokens, tokens, Q_SIGMA20, device)
            V = gauss_i8(seed, tid(g, ROLE_V), tokens, head_dim, Q_SIGMA20, device)
            out.append(Problem(f"L{layer}.h{h}.pv", P, V, exact_matmul_i32(P, V), 2 * g + 1))
    return out


def problem_bytes(problems: List[Problem]) -> int:
    """Algorithmic HBM bytes of one proving pass: every input element read exactly once."""
    return sum(p.A.numel() + p.B.numel() + 4 * p.C.numel() for p in problems)


def prover_field_macs(problems: List[Problem]) -> int:
    """Field multiply-accumulates the prover executes: m*k + k*n + m*n + 5 * 2^ceil(log2 k)."""
    total = 0
    for p in problems:
        m, k, n = p.mkn
        total += m * k + k * n + m * n + 5 * (1 << max(0, (k - 1).bit_length()))
    return total


def proved_matmul_macs(problems: List[Problem]) -> int:
    return sum(m * k * n for (m, k, n) in (p.mkn for p in problems))


# ---------------------------------------------------------------------------- logits for the LDD


ROLE_LOGIT, ROLE_LOGIT_NOISE, ROLE_LOGIT_HOT = 16, 17, 18
LOGIT_SCALE = 2.5 / 209.02           # byte sums have standard deviation ~209: bulk logits ~ N(0, 2.5^2)
HOT_TOKENS = 12                      # entries per row lifted well above the bulk (the plausible next tokens)

# deployment regimes, as noise added to the reference logits (standard deviation of the noise):
# a benign reduced-precision run, an aggressive quantisation, and a different model altogether
NOISE_BENIGN, NOISE_QUANTISED = 0.02, 0.25


def reference_logits(seed: int, steps: int, vocab: int, device="cpu", group: int = 0) -> torch.Tensor:
    """float32 logits (steps x vocab): an approx-Gaussian bulk plus HOT_TOKENS boosted entries per
    row.  Built from integers and one float32 multiply, so CPU and CUDA give identical bits."""
    s = _fill(seed, tid(group, ROLE_LOGIT), steps, vocab, device, lambda u: byte_sum(u) - 1020, dtype=torch.int32).to(torch.int64)
    idx = torch.arange(steps * HOT_TOKENS, dtype=torch.int64, device=device)
    u = stream_u64(seed, tid(group, ROLE_LOGIT_HOT), idx)
    col = ((_lsr(u, 32) * vocab) >> 32).view(steps, HOT_TOKENS)                 # hot token index in [0, vocab)
    lift = (700 + 60 * (HOT_TOKENS - torch.arange(HOT_TOKENS, device=device, dtype=torch.int64))).expand(steps, -1)
    s.scatter_add_(1, col, lift.contiguous())                                   # integer adds: order-independent
    return (s.to(torch.float32) * LOGIT_SCALE).contiguous()


def deployed_logits(ref: torch.Tensor, seed: int, noise: float, group: int = 0) -> torch.Tensor:
    """Reference logits plus seeded approx-Gaussian noise of standard deviation ``noise`` (two separately
    rounded float32 operations per entry: identical bits on CPU and CUDA)."""
    steps, vocab = ref.shape
    z = _fill(seed, tid(group, ROLE_LOGIT_NOISE), steps, vocab, ref.device, lambda u: byte_sum(u) - 1020, dtype=torch.int32)
    scaled = z.to(torch.float32) * (noise / 209.02)
    return (ref + scaled).contiguous()


def request_offsets(seed: int, steps: int, requests: int, device="cpu") -> torch.Tensor:
    """int64 offsets (requests + 1) cutting ``steps`` decision steps into requests of seeded ragged lengths."""
    idx = torch.arange(max(requests - 1, 0), dtype=torch.int64, device="cpu")
    cuts = ((_lsr(stream_u64(seed, tid(0, ROLE_ROUTER), idx), 32) * (steps + 1)) >> 32).sort().values
    out = torch.cat([torch.zeros(1, dtype=torch.int64), cuts, torch.full((1,), steps, dtype=torch.int64)])
    return out.to(device)
