"""Seeded synthetic inputs for the five benchmark configurations.

This module holds input generation only: random draws, casts to fp16, planted rows. It contains none
of the method's arithmetic and is the only code shared by the oracle-side tests and the CUDA-side
tests. Quaternions are drawn as 4 iid N(0,1) components and scaled to unit length (Haar measure on
S^3): that is the input distribution, both implementations renormalise on their own.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

SEED0 = 260808081
# stream ids
K_STREAM, V_STREAM, Q_STREAM, QUAT_STREAM, STRUCT_STREAM, STEP_STREAM = range(6)


def stream_seed(config: int, k: int) -> int:
    return SEED0 + 1000 * config + k


def rng(config: int, k: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(stream_seed(config, k)))


def to_fp16(a: np.ndarray) -> np.ndarray:
    return np.clip(a, -65504.0, 65504.0).astype(np.float16)


def cap128(rows: int) -> int:
    """Cache capacity for `rows` rows: the next multiple of 128 (the V side is stored in 128-row blocks)."""
    return ((int(rows) + 127) // 128) * 128


def quaternion_pairs(gen: np.random.Generator, n_kv_heads: int, d: int) -> np.ndarray:
    """[H_kv][d/4][8] fp32 = (q_L.wxyz, q_R.wxyz), each quaternion of unit length."""
    q = gen.standard_normal((n_kv_heads, d // 4, 2, 4))
    q /= np.linalg.norm(q, axis=-1, keepdims=True)
    return q.reshape(n_kv_heads, d // 4, 8).astype(np.float32)


@dataclass
class Workload:
    name: str
    B: int
    H_q: int
    H_kv: int
    d: int
    t_cap: int               # cache rows per (sequence, KV head): multiple of 128, >= T
    k: np.ndarray            # fp16 [B][T][H_kv][d]
    v: np.ndarray            # fp16 [B][T][H_kv][d]
    q: np.ndarray            # fp16 [B][H_q][d]
    quats: np.ndarray        # fp32 [H_kv][d/4][8]
    seq_lens: np.ndarray     # int32 [B] rows of k/v that are valid
    extra: dict = field(default_factory=dict)

    @property
    def G(self) -> int:
        return self.H_q // self.H_kv


def _outlier_channels(gen, x, n=4, factor=20.0):
    d = x.shape[-1]
    ch = gen.choice(d, size=n, replace=False)
    x[..., ch] *= factor
    return ch


def config1(T: int = 1024, H_q: int = 4, H_kv: int = 1, d: int = 128, cfg: int = 1) -> Workload:
    """Tiny decode: N(0,1) K/V with 4 outlier channels x20 (drawn separately for K and V), q N(0,1)."""
    k = rng(cfg, K_STREAM).standard_normal((1, T, H_kv, d))
    v = rng(cfg, V_STREAM).standard_normal((1, T, H_kv, d))
    sg = rng(cfg, STRUCT_STREAM)
    kch = _outlier_channels(sg, k)
    vch = _outlier_channels(sg, v)
    q = rng(cfg, Q_STREAM).standard_normal((1, H_q, d))
    return Workload("config1", 1, H_q, H_kv, d, cap128(T), to_fp16(k), to_fp16(v), to_fp16(q),
                    quaternion_pairs(rng(cfg, QUAT_STREAM), H_kv, d), np.array([T], np.int32),
                    dict(k_outliers=kch, v_outliers=vch))


def config2(T: int = 8192, steps: int = 64, H_q: int = 32, H_kv: int = 4, d: int = 128) -> Workload:
    """~30B-A3B-shaped attention: per-(head, channel) log-normal scales (sigma 1), prefill then decode steps."""
    cfg = 2
    sg = rng(cfg, STRUCT_STREAM)
    ks = np.exp(sg.standard_normal((1, 1, H_kv, d)))
    vs = np.exp(sg.standard_normal((1, 1, H_kv, d)))
    k = rng(cfg, K_STREAM).standard_normal((1, T, H_kv, d)) * ks
    v = rng(cfg, V_STREAM).standard_normal((1, T, H_kv, d)) * vs
    q = rng(cfg, Q_STREAM).standard_normal((1, H_q, d))
    st = rng(cfg, STEP_STREAM)
    step_k = st.standard_normal((steps, 1, 1, H_kv, d)) * ks
    step_v = st.standard_normal((steps, 1, 1, H_kv, d)) * vs
    step_q = st.standard_normal((steps, 1, H_q, d))
    return Workload("config2", 1, H_q, H_kv, d, cap128(T + steps), to_fp16(k), to_fp16(v), to_fp16(q),
                    quaternion_pairs(rng(cfg, QUAT_STREAM), H_kv, d), np.array([T], np.int32),
                    dict(step_k=to_fp16(step_k), step_v=to_fp16(step_v), step_q=to_fp16(step_q), steps=steps))


def config3(T: int = 16384, H_q: int = 16, H_kv: int = 8, d: int = 256) -> Workload:
    """Wider heads: 0.5 x Student-t(nu=3) K/V."""
    cfg = 3
    k = 0.5 * rng(cfg, K_STREAM).standard_t(3.0, (1, T, H_kv, d))
    v = 0.5 * rng(cfg, V_STREAM).standard_t(3.0, (1, T, H_kv, d))
    q = rng(cfg, Q_STREAM).standard_normal((1, H_q, d))
    return Workload("config3", 1, H_q, H_kv, d, cap128(T), to_fp16(k), to_fp16(v), to_fp16(q),
                    quaternion_pairs(rng(cfg, QUAT_STREAM), H_kv, d), np.array([T], np.int32))


def config4(T: int = 32768, H_q: int = 32, H_kv: int = 8, d: int = 128) -> Workload:
    """Long-context synthetic retrieval: Gaussian K/V; one needle per query head at a distinct seeded
    position p_h: k[p_h] = 4 * q_h (in the head's KV head), v[p_h] = 8 * e_{c_h} with distinct channels c_h."""
    cfg = 4
    k = to_fp16(rng(cfg, K_STREAM).standard_normal((1, T, H_kv, d)))
    v = to_fp16(rng(cfg, V_STREAM).standard_normal((1, T, H_kv, d)))
    q = to_fp16(rng(cfg, Q_STREAM).standard_normal((1, H_q, d)))
    sg = rng(cfg, STRUCT_STREAM)
    pos = sg.choice(T, size=H_q, replace=False).astype(np.int64)
    chan = sg.choice(d, size=H_q, replace=False).astype(np.int64)
    G = H_q // H_kv
    for h in range(H_q):
        g = h // G
        k[0, pos[h], g, :] = to_fp16(4.0 * q[0, h, :].astype(np.float64))
        v[0, pos[h], g, :] = 0
        v[0, pos[h], g, chan[h]] = 8.0
    return Workload("config4", 1, H_q, H_kv, d, cap128(T), k, v, q, quaternion_pairs(rng(cfg, QUAT_STREAM), H_kv, d),
                    np.array([T], np.int32), dict(needle_pos=pos, needle_chan=chan))


def config5_lengths(B: int, ctx: int) -> np.ndarray:
    """Ragged per-sequence lengths floor(ctx * U[0.5, 1.0])."""
    sg = np.random.Generator(np.random.Philox(stream_seed(5, STRUCT_STREAM) + 17 * B + ctx))
    return np.floor(ctx * sg.uniform(0.5, 1.0, size=B)).astype(np.int32)


def config5(B: int, ctx: int, H_q: int = 64, H_kv: int = 8, d: int = 128) -> Workload:
    """Batched serving point (host generation; use config5_device for the large points)."""
    cfg = 5
    lens = config5_lengths(B, ctx)
    sub = 100 * B + ctx // 1024
    k = np.random.Generator(np.random.Philox(stream_seed(cfg, K_STREAM) + sub)).standard_normal((B, ctx, H_kv, d))
    v = np.random.Generator(np.random.Philox(stream_seed(cfg, V_STREAM) + sub)).standard_normal((B, ctx, H_kv, d))
    sg = np.random.Generator(np.random.Philox(stream_seed(cfg, STRUCT_STREAM) + sub))
    kch = _outlier_channels(sg, k)
    vch = _outlier_channels(sg, v)
    q = np.random.Generator(np.random.Philox(stream_seed(cfg, Q_STREAM) + sub)).standard_normal((B, H_q, d))
    return Workload(f"config5_B{B}_ctx{ctx}", B, H_q, H_kv, d, cap128(ctx), to_fp16(k), to_fp16(v), to_fp16(q),
                    quaternion_pairs(rng(cfg, QUAT_STREAM), H_kv, d), lens, dict(k_outliers=kch, v_outliers=vch))


def config5_device(B: int, ctx: int, device, H_q: int = 64, H_kv: int = 8, d: int = 128, chunk_seqs: int = 4,
                   full_lengths: bool = False):
    """Generator of the large serving points on the GPU (seeded torch generator): yields, per chunk of
    sequences, (b0, k, v) fp16 device tensors [nb][ctx][H_kv][d]; also returns q, lengths and quaternions.
    full_lengths: every sequence holds ctx rows (a stack of per-layer caches instead of a ragged batch)."""
    import torch

    cfg = 5
    lens = np.full(B, ctx, np.int32) if full_lengths else config5_lengths(B, ctx)
    sub = 100 * B + ctx // 1024
    sg = np.random.Generator(np.random.Philox(stream_seed(cfg, STRUCT_STREAM) + sub))
    kch = sg.choice(d, size=4, replace=False)
    vch = sg.choice(d, size=4, replace=False)
    gen = torch.Generator(device=device)
    gen.manual_seed(stream_seed(cfg, K_STREAM) + sub)
    q = torch.randn((B, H_q, d), generator=gen, device=device, dtype=torch.float32).to(torch.float16)
    quats = quaternion_pairs(rng(cfg, QUAT_STREAM), H_kv, d)

    def chunks():
        for b0 in range(0, B, chunk_seqs):
            nb = min(chunk_seqs, B - b0)
            k = torch.randn((nb, ctx, H_kv, d), generator=gen, device=device, dtype=torch.float32)
            k[..., torch.as_tensor(kch, device=device)] *= 20.0
            v = torch.randn((nb, ctx, H_kv, d), generator=gen, device=device, dtype=torch.float32)
            v[..., torch.as_tensor(vch, device=device)] *= 20.0
            yield b0, k.to(torch.float16), v.to(torch.float16)

    return dict(q=q, lens=lens, quats=quats, chunks=chunks, B=B, ctx=ctx, H_q=H_q, H_kv=H_kv, d=d)


def tiny(seed: int, B: int, H_q: int, H_kv: int, d: int, T: int, lens=None, scale: float = 1.0) -> Workload:
    """Small Gaussian case for brute-force checks and shape sweeps."""
    g = np.random.Generator(np.random.Philox(SEED0 + 7919 * seed))
    k = to_fp16(scale * g.standard_normal((B, T, H_kv, d)))
    v = to_fp16(scale * g.standard_normal((B, T, H_kv, d)))
    q = to_fp16(g.standard_normal((B, H_q, d)))
    quats = quaternion_pairs(g, H_kv, d)
    if lens is None:
        lens = np.full(B, T, np.int32)
    return Workload(f"tiny{seed}", B, H_q, H_kv, d, cap128(T), k, v, q, quats, np.asarray(lens, np.int32))
