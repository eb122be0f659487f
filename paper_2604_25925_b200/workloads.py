"""Seeded synthetic verify-step inputs (shared by the tests, the smoke check and the benchmark).

This module only *makes inputs*: logits shaped like language-model outputs, draft tokens drawn
from the draft rows, and pre-drawn uniforms.  It contains none of the verification arithmetic
(no softmax, no coupling sums, no acceptance weights): draft tokens are drawn with the
Gumbel-max trick, i.e. ``argmax_x(z_x / T + Gumbel)``, which samples softmax(z/T) without ever
forming it.

Randomness is a counter-based hash (splitmix64 finaliser on int64 tensors), so a value depends
only on (seed, row key, vocabulary index) and the same code runs on CPU and CUDA tensors.

Recipe (stand-in for the paper's language-model workloads, whose weights and datasets are not
available):
  target row  z_q[x] = sigma * N(0,1) + boost * rank(x)^(-1.1)   (rank: a random permutation per row)
  draft row   z_p[x] = alpha * z_q[x] + sqrt(1 - alpha^2) * sigma * N'(0,1)
A row is keyed by the token prefix it is conditioned on, so all K drafts of a batch row share the
position-0 rows and two drafts with equal prefixes share their rows, as they would for a real
model.  Draft tokens are i.i.d. across drafts (noise keyed by (b, k, i)).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

_GOLD = -7046029254386353131          # 0x9E3779B97F4A7C15 as int64
_M1 = -4658895280553007687            # 0xBF58476D1CE4E5B9
_M2 = -7723592293110705685            # 0x94D049BB133111EB


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    B: int
    K: int
    gamma: int
    V: int
    dtype: str = "fp32"        # "fp32" or "bf16" (storage type of the logits)
    temperature: float = 1.0
    alpha: float = 0.85        # draft/target logit correlation
    sigma: float = 2.0         # std of the Gaussian part
    boost: float = 6.0         # Zipf rank boost amplitude (0 = none)
    zipf_s: float = 1.1
    seed: int = 1234
    consistent_prefix: bool = True

    def logit_bytes(self) -> int:
        s = 2 if self.dtype == "bf16" else 4
        return (self.B * self.K * (2 * self.gamma + 1) * self.V) * s


CONFIGS = {
    # tiny case for enumeration / Monte-Carlo checks
    "c1": VerifyConfig("c1", B=1, K=2, gamma=3, V=16, alpha=0.8, sigma=1.5, boost=0.0, seed=1234),
    "c2": VerifyConfig("c2", B=8, K=4, gamma=4, V=32000, alpha=0.85, seed=1235),
    "c3": VerifyConfig("c3", B=32, K=4, gamma=5, V=128256, dtype="bf16", temperature=0.7,
                       alpha=0.7, seed=1236),
    "c4": VerifyConfig("c4", B=64, K=8, gamma=8, V=151936, alpha=0.9, seed=1237),
    # the paper's own operating points (Table 2): one prompt, K = 3 drafts, L = 12 or 8, T = 0.4,
    # a 32k vocabulary (DeepSeek-coder's 32256)
    "paper_l12": VerifyConfig("paper_l12", B=1, K=3, gamma=12, V=32256, temperature=0.4, alpha=0.85, seed=1240),
    "paper_l8": VerifyConfig("paper_l8", B=1, K=3, gamma=8, V=32256, temperature=0.4, alpha=0.85, seed=1241),
    # the longest draft length of the paper's sweep over L
    "paper_l24": VerifyConfig("paper_l24", B=1, K=3, gamma=24, V=32256, temperature=0.4, alpha=0.85, seed=1242),
}


def sweep_c5():
    """The B=256, gamma=4, V=32000 sweep over K x alpha x temperature."""
    pts = []
    for K in (1, 2, 4, 8):
        for alpha in (0.5, 0.8, 0.95):
            for T in (0.6, 1.0):
                pts.append(VerifyConfig(f"c5_K{K}_a{alpha}_T{T}", B=256, K=K, gamma=4, V=32000,
                                        alpha=alpha, temperature=T, seed=1238))
    return pts


def get_config(name: str) -> VerifyConfig:
    """A named configuration (c1..c4, c5_K*_a*_T*), or a spec such as
    ``B=8,K=8,gamma=8,V=151936,dtype=fp32,T=1.0,alpha=0.9`` (omitted fields keep their defaults)."""
    if name in CONFIGS:
        return CONFIGS[name]
    for c in sweep_c5():
        if c.name == name:
            return c
    if "=" in name:
        alias = {"T": "temperature", "g": "gamma"}
        kinds = {"B": int, "K": int, "gamma": int, "V": int, "dtype": str, "temperature": float,
                 "alpha": float, "sigma": float, "boost": float, "zipf_s": float, "seed": int}
        fields = {"B": 8, "K": 4, "gamma": 4, "V": 32000}
        for part in name.split(","):
            k, v = part.split("=")
            k = alias.get(k.strip(), k.strip())
            fields[k] = kinds[k](v.strip())
        return VerifyConfig(name.replace(" ", ""), **fields)
    raise KeyError(name)


# ---------------------------------------------------------------- counter-based randomness
def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    x = x + _GOLD
    x = (x ^ _lsr(x, 30)) * _M1
    x = (x ^ _lsr(x, 27)) * _M2
    return x ^ _lsr(x, 31)


def _key(*parts) -> torch.Tensor:
    """Fold integer tensors / ints into one int64 key tensor (broadcasting)."""
    k = None
    for p in parts:
        if not torch.is_tensor(p):
            p = torch.tensor(int(p), dtype=torch.int64)
        p = p.to(torch.int64)
        k = _mix(p) if k is None else _mix(k ^ (_mix(p) * _M1))
    return k


def _u24(bits: torch.Tensor) -> torch.Tensor:
    """float32 uniform in [0,1) with 24 random bits."""
    return _lsr(bits, 40).to(torch.float32) * (1.0 / 16777216.0)


def _normal(key: torch.Tensor, x: torch.Tensor, stream: int) -> torch.Tensor:
    """Standard normal per (key, x): Box-Muller on two hashed uniforms. key [R,1], x [1,V]."""
    h1 = _mix((key + x * _GOLD) ^ (stream + 1))
    u1 = 1.0 - _u24(h1)                                      # (0,1]
    u2 = _u24(_mix(h1))
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(6.283185307179586 * u2)


def _rows(cfg: VerifyConfig, key: torch.Tensor, device) -> tuple[torch.Tensor, torch.Tensor]:
    """Target and draft logit rows [R, V] (float32) for row keys [R]."""
    V = cfg.V
    x = torch.arange(V, dtype=torch.int64, device=device).unsqueeze(0)
    k = key.to(device).unsqueeze(1)
    zq = cfg.sigma * _normal(k, x, 0)
    if cfg.boost != 0.0:
        order = torch.argsort(_lsr(_mix((k + x * _GOLD) ^ 0x5A17), 1), dim=1)
        ranks = torch.arange(1, V + 1, dtype=torch.float32, device=device)
        b = (cfg.boost * ranks.pow(-cfg.zipf_s)).unsqueeze(0).expand(order.shape[0], V)
        zq = zq + torch.zeros_like(zq).scatter_(1, order, b)
        del order, b
    noise = _normal(k, x, 1)
    zp = cfg.alpha * zq + (1.0 - cfg.alpha * cfg.alpha) ** 0.5 * cfg.sigma * noise
    return zq, zp


def _gumbel(key: torch.Tensor, V: int, device) -> torch.Tensor:
    x = torch.arange(V, dtype=torch.int64, device=device).unsqueeze(0)
    u = _u24(_mix((key.to(device).unsqueeze(1) + x * _GOLD) ^ 0x6B43)).clamp_min(2.0 ** -25)
    return -torch.log(-torch.log(u))


@dataclass
class VerifyInputs:
    cfg: VerifyConfig
    target_logits: torch.Tensor   # [B,K,gamma+1,V] float32 or bfloat16
    draft_logits: torch.Tensor    # [B,K,gamma,V]
    draft_tokens: torch.Tensor    # [B,K,gamma] int32
    uniforms: torch.Tensor        # [B,K*gamma+1] float32 in [0,1)

    def to(self, device) -> "VerifyInputs":
        return VerifyInputs(self.cfg, self.target_logits.to(device), self.draft_logits.to(device),
                            self.draft_tokens.to(device), self.uniforms.to(device))


def make_uniforms(B: int, K: int, gamma: int, seed: int, device="cpu", draw: int = 0) -> torch.Tensor:
    """[B, K*gamma+1] float32 U[0,1): eta for trial (k,i) at k*gamma+(i-1), the sampling uniform last."""
    n = K * gamma + 1
    b = torch.arange(B, dtype=torch.int64, device=device).unsqueeze(1)
    j = torch.arange(n, dtype=torch.int64, device=device).unsqueeze(0)
    return _u24(_mix(_key(seed, 0x0E7A, draw).to(device) + b * _GOLD + j * _M1)).contiguous()


def make_inputs(cfg: VerifyConfig, device="cpu", set_index: int = 0,
                row_batch: int = 256) -> VerifyInputs:
    """Build one seeded input set. ``set_index`` varies the seed (rotating benchmark sets)."""
    B, K, g, V = cfg.B, cfg.K, cfg.gamma, cfg.V
    seed = cfg.seed + 7919 * set_index
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    zq_all = torch.empty((B, K, g + 1, V), dtype=dt, device=device)
    zp_all = torch.empty((B, K, g, V), dtype=dt, device=device)
    tok = torch.empty((B, K, g), dtype=torch.int32, device=device)
    bidx = torch.arange(B, dtype=torch.int64).unsqueeze(1).expand(B, K)
    kidx = torch.arange(K, dtype=torch.int64).unsqueeze(0).expand(B, K)
    if cfg.consistent_prefix:
        key = _key(seed, bidx)                       # position-0 rows shared by all drafts
    else:
        key = _key(seed, bidx, kidx)
    key = key.reshape(-1)                            # [B*K]
    R = B * K
    for i in range(g + 1):
        gkey = _key(seed, 0x7A11, bidx, kidx, i).reshape(-1)
        for r0 in range(0, R, row_batch):
            r1 = min(R, r0 + row_batch)
            zq, zp = _rows(cfg, key[r0:r1], device)
            zq_s = zq.to(dt)
            zq_all.view(R, g + 1, V)[r0:r1, i] = zq_s
            if i < g:
                zp_s = zp.to(dt)
                zp_all.view(R, g, V)[r0:r1, i] = zp_s
                score = zp_s.to(torch.float32) / cfg.temperature + _gumbel(gkey[r0:r1], V, device)
                tok.view(R, g)[r0:r1, i] = torch.argmax(score, dim=1).to(torch.int32)
            del zq, zp
        if i < g:
            t = tok.view(R, g)[:, i].to("cpu", torch.int64)
            if cfg.consistent_prefix:
                key = _mix(key ^ ((t + 1) * _M2))
            else:
                key = _key(key, i + 1)
    u = make_uniforms(B, K, g, seed, device)
    return VerifyInputs(cfg, zq_all, zp_all, tok, u)


def with_batch(cfg: VerifyConfig, B: int) -> VerifyConfig:
    return replace(cfg, B=B)
