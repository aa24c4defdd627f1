"""Seeded synthetic inputs for the expert-cached MoE layer.

This module only *draws inputs*: expert-weight records, router logits and
activations.  It contains none of the layer's arithmetic (no routing, no cache
logic, no FFN, no dequantisation) so that the CPU oracle and the CUDA library
can both be fed from it without sharing any of the method's code.  Everything
is a pure function of an integer seed.

Expert record formats (one contiguous record per (layer, expert); the pool is
``n_layers * n_experts`` records back to back, record index ``l * E + e``, the
flattened identifier of Sec. 4.2 of the paper):

``bf16``  ``I/16`` units of 16 neurons, each ``96*d`` bytes: a gate part, an up part and a
          down part of ``32*d`` bytes each.  Gate/up part: tiles of 16 neurons x 32 hidden
          indices (1 KiB), tile ``i // 32``; a tile is two groups of 8 neuron rows of 64 bytes
          (group ``(n % 16) // 8``, row ``r = n % 8``); the four 16-byte chunks of a row are
          stored swizzled: chunk ``(i % 32) // 8`` sits at position ``chunk ^ (r >> 1)``.
          Down part: tiles of 16 output columns x the unit's 16 neurons (512 bytes), tile
          ``c // 16``; two groups of 8 column rows of 32 bytes (group ``(c % 16) // 8``,
          row ``r = c % 8``); the two 16-byte chunks of a row are stored at position
          ``((n % 16) // 8) ^ (r >> 2)``.  ``S = 3*I*d*2`` bytes.
``int4``  4-bit two's-complement codes in [-8, 7] and bf16 scales, weight = scale * code, groups of
          128 along the contraction dimension (``G = d/128`` hidden groups for gate/up, ``NG = I/128``
          neuron groups for down), in tensor-core tile order.  Three sections:
          A. ``I/16`` units of 16 neurons, ``2112*G`` bytes each: gate tiles, up tiles, gate scales, up
             scales.  A tile is 16 neuron rows x 128 hidden indices = 16 rows of 64 bytes; in a row the
             code of hidden index ``128*grp + 32*j + 8*q + e`` is nibble ``e`` (low nibble = even ``e``) of
             the little-endian 32-bit word ``j`` of the 16-byte chunk ``q``.  The scales of a tile are 8
             pairs ``(row r, row r+8)`` of bf16.
          B. down codes: for each column block ``cb`` (``CBW = 64*min(16, d/64)`` columns), neuron group
             ``ng`` and 16-neuron step ``uu`` of the group: ``CBW/64`` x 512 bytes; in each 512 bytes lane
             ``l = 4g + q`` owns 16 bytes = 4 words, word ``j`` belongs to the 16-column tile ``4w + j`` of the
             block; its nibble ``e`` is the code of column ``g + 8*(e & 1)`` of the tile and neuron
             ``4q + e // 2`` of the step.
          C. down scales ``sd[ng][column]`` in the order (ng, cb, w, g, j, half): 8 pairs per tile again.
          ``S = 3*I*d/2 + (2*I*d/128 + (I/128)*d)*2``.
``mxfp4`` 4-bit e2m1 codes (bit 3 sign; bits 2..0 index 0, 0.5, 1, 1.5, 2, 3, 4, 6) with one power-of-two scale byte
          ``b`` (value ``2**(b - 127)``) per block of 32 consecutive elements along the contraction dimension
          (the OCP microscaling FP4 element and scale formats).  The code sections are those of ``int4``; the scales:
          A. per tile 64 bytes after the tiles of a unit (``2176*G`` bytes per unit): for ``r`` in 0..7 the four block
             scales (``j`` = 0..3) of row ``r``, then those of row ``r+8``.
          C. order (ng, cb, w, g, j, half, m): per lane ``g`` 32 bytes = for each tile ``j`` and column half the four
             32-neuron blocks ``m`` of the 128-neuron group.
          ``S = 3*I*d/2 + 3*I*d/32``.
``mxfp4tc`` the ``mxfp4`` numbers as operand images of the block-scaled tensor-core instruction (K-major core
          matrices of 8 rows x 16 bytes, scale factors in groups of 128 rows x 4 blocks).  Section A: per (group of
          128 neurons, 128 hidden indices) 17408 bytes = gate image, up image (8192 each), gate scales, up scales (512
          each); section B: per (group of 128 output columns, 128 neurons) 8704 bytes = image, scales.  Byte of (row
          ``r``, index ``k`` < 128) in an image: ``4096*(k//64) + 2048*((k%64)//32) + 128*(r//8) + 16*(r%8) +
          (k%32)//2`` (low nibble = even ``k``); scale of (row ``r``, block ``b``): ``16*(r%32) + 4*(r//32) + b``.
          ``S`` as for ``mxfp4``.
``nvfp4`` the same e2m1 codes with one unsigned e4m3 scale byte per block of 16 consecutive elements along the
          contraction dimension and one float32 scale per matrix.  Differences from ``mxfp4``:
          A. ``2304*G`` bytes per unit; in a gate/up tile row the code of hidden index ``128*grp + 32*j + 16*(e & 1)
             + 4*q + e // 2`` is nibble ``e`` of word ``j`` of chunk ``q`` (so that the even nibbles of a word row
             are one scale block and the odd nibbles the next); per tile 128 scale bytes: for ``r`` in 0..7 the
             eight block scales of row ``r``, then those of row ``r+8``.
          C. order (ng, cb, w, g, j, half, unit): per lane ``g`` 64 bytes = for each tile ``j`` and column half the
             eight 16-neuron blocks of the 128-neuron group.
          Then the three matrix scales (gate, up, down) as float32, zero-padded to 256 bytes.
          ``S = 3*I*d/2 + 3*I*d/16 + 256``.

The routing-logit recipes follow the workload descriptions: a Zipf-style
popularity bias ``b_e = -alpha * ln(rank_e)`` with ``rank`` a seeded permutation
of ``1..E`` per layer, and an AR(1) chain per (layer, batch row) with unit
stationary variance, ``u_t = rho*u_{t-1} + sqrt(1-rho^2)*eps_t``, ``z_t = u_t + b``.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch

GROUP = 128  # int4 quantisation group length along the contraction dimension
MX_BLOCK = 32  # elements that share one scale byte in the mxfp4 records
NV_BLOCK = 16  # elements that share one e4m3 scale byte in the nvfp4 records
NV_TAIL = 256  # bytes of the record's tail holding the three float32 matrix scales


@dataclasses.dataclass(frozen=True)
class LayerShape:
    d: int            # hidden size
    inter: int        # expert intermediate size I
    n_experts: int    # routed experts E
    top_k: int
    wdtype: str = "bf16"   # "bf16" | "int4" | "mxfp4" | "mxfp4tc" | "nvfp4"
    n_shared: int = 0      # always-resident shared experts (0 or 1)

    @property
    def expert_bytes(self) -> int:
        if self.wdtype == "bf16":
            return 3 * self.inter * self.d * 2
        if self.wdtype == "int4":
            payload = 3 * self.inter * self.d // 2
            scales = (2 * self.inter * (self.d // GROUP) + (self.inter // GROUP) * self.d) * 2
            return payload + scales
        if self.wdtype in ("mxfp4", "mxfp4tc"):
            return 3 * self.inter * self.d // 2 + 3 * self.inter * self.d // MX_BLOCK
        if self.wdtype == "nvfp4":
            return 3 * self.inter * self.d // 2 + 3 * self.inter * self.d // NV_BLOCK + NV_TAIL
        raise ValueError(self.wdtype)


# The shapes of the five workload configurations.
TINY = LayerShape(d=256, inter=128, n_experts=8, top_k=2)
QWEN3_30B = LayerShape(d=2048, inter=768, n_experts=128, top_k=8)
DSV3_INT4 = LayerShape(d=7168, inter=2048, n_experts=256, top_k=8, wdtype="int4", n_shared=1)
DSV3_MXFP4 = LayerShape(d=7168, inter=2048, n_experts=256, top_k=8, wdtype="mxfp4", n_shared=1)
DSV3_MXFP4TC = LayerShape(d=7168, inter=2048, n_experts=256, top_k=8, wdtype="mxfp4tc", n_shared=1)
DSV3_NVFP4 = LayerShape(d=7168, inter=2048, n_experts=256, top_k=8, wdtype="nvfp4", n_shared=1)


def mix64(*vals: int) -> int:
    """splitmix64-style mix of a tuple of small integers into one 63-bit seed."""
    h = 0x9E3779B97F4A7C15
    for v in vals:
        h = (h ^ (int(v) & 0xFFFFFFFFFFFFFFFF)) & 0xFFFFFFFFFFFFFFFF
        h = (h + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
        h = ((h ^ (h >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        h = ((h ^ (h >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
        h ^= h >> 31
    return h & 0x7FFFFFFFFFFFFFFF


_TAG_W, _TAG_RANK, _TAG_U0, _TAG_EPS, _TAG_X, _TAG_LOGIT = 1, 2, 3, 4, 5, 6


def slots_for_fraction(frac: float, n_experts: int) -> int:
    """Cache fraction -> slots per layer (rounded up)."""
    return int(math.ceil(frac * n_experts - 1e-9))


# --------------------------------------------------------------------------
# expert weights
# --------------------------------------------------------------------------

def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _quantise_int4(w: torch.Tensor, group_axis: int) -> tuple[torch.Tensor, torch.Tensor]:
    """Symmetric int4 quantiser used to *produce* the synthetic pool.

    ``w``: fp32 ``[n, I, d]``; groups of 128 along ``group_axis`` (1 or 2).
    Returns (codes int8 in [-8,7] with w's shape, scales bf16 with the group
    axis reduced by 128).
    """
    n, I, d = w.shape
    if group_axis == 2:
        wg = w.reshape(n, I, d // GROUP, GROUP)
        amax = wg.abs().amax(dim=3)                              # [n, I, d/128]
        scale = (amax / 7.0).to(torch.bfloat16)
        sf = scale.to(torch.float32).unsqueeze(3)
        q = torch.where(sf > 0, torch.round(wg / torch.where(sf > 0, sf, torch.ones_like(sf))),
                        torch.zeros_like(wg))
        q = q.clamp_(-8, 7).reshape(n, I, d)
    else:
        wg = w.reshape(n, I // GROUP, GROUP, d)
        amax = wg.abs().amax(dim=2)                              # [n, I/128, d]
        scale = (amax / 7.0).to(torch.bfloat16)
        sf = scale.to(torch.float32).unsqueeze(2)
        q = torch.where(sf > 0, torch.round(wg / torch.where(sf > 0, sf, torch.ones_like(sf))),
                        torch.zeros_like(wg))
        q = q.clamp_(-8, 7).reshape(n, I, d)
    return q.to(torch.int8), scale


def _pack_nibbles(q: torch.Tensor) -> torch.Tensor:
    """int8 codes ``[..., n]`` -> uint8 ``[..., n/2]``, low nibble = even index."""
    u = (q.to(torch.int16) & 0xF).to(torch.uint8)
    return u[..., 0::2] | (u[..., 1::2] << 4)


def _quantise_mxfp4(w: torch.Tensor, block_axis: int) -> tuple[torch.Tensor, torch.Tensor]:
    """Microscaling FP4 quantiser used to *produce* the synthetic pool.

    ``w``: fp32 ``[I, d]``; blocks of 32 along ``block_axis`` (0 or 1).  Returns (codes uint8 in 0..15 with w's
    shape, scale bytes uint8 with the block axis reduced by 32).  Shared exponent = floor(log2(amax)) - 2 (2 = the
    exponent of the largest e2m1 magnitude), elements rounded to the nearest e2m1 value (ties to the even code),
    saturating at 6.
    """
    I, d = w.shape
    wb = w.reshape(I, d // MX_BLOCK, MX_BLOCK) if block_axis == 1 else w.reshape(I // MX_BLOCK, MX_BLOCK, d)
    ax = 2 if block_axis == 1 else 1
    amax = wb.abs().amax(dim=ax, keepdim=True)
    e = torch.floor(torch.log2(torch.where(amax > 0, amax, torch.ones_like(amax)))) - 2
    b = torch.clamp(e + 127, 0, 254)
    v = wb / torch.exp2(b - 127)
    a = v.abs().clamp(max=6.0)
    bounds = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], device=w.device, dtype=torch.float32)
    lo_ = torch.bucketize(a, bounds, right=False)     # bounds strictly below a
    hi_ = torch.bucketize(a, bounds, right=True)      # bounds at or below a
    idx = torch.where(lo_ != hi_, torch.where(lo_ % 2 == 0, lo_, hi_), lo_)   # a tie goes to the even code
    code = (idx | torch.where(v < 0, 8, 0)).to(torch.uint8)
    return code.reshape(I, d), b.squeeze(ax).to(torch.uint8)


def _pack_mxfp4_record(cg, cu, cd, bg, bu, bd) -> torch.Tensor:
    """Codes uint8 ``[I][d]`` (gate/up: one row per neuron; down: ``[n][c]``), scale bytes ``bg, bu [I][d/32]``,
    ``bd [I/32][d]`` -> the tiled record, uint8 flat."""
    I, d = cg.shape
    dev = cg.device
    U, G, NG = I // 16, d // GROUP, I // GROUP
    nwd = min(16, d // 64)
    cbw = 64 * nwd
    CB = d // cbw

    def gu_tiles(c):      # [U][16 rows][G][j][q][e] -> [U][G][row][q][j][e], nibbles packed along e
        t = c.reshape(U, 16, G, 4, 4, 8).permute(0, 2, 1, 4, 3, 5)
        return (t[..., 0::2] | (t[..., 1::2] << 4)).reshape(U, G * 1024)

    def gu_scales(b_):    # [U][half][r][G][j] -> [U][G][r][half][j]
        return b_.reshape(U, 2, 8, G, 4).permute(0, 3, 2, 1, 4).reshape(U, G * 64)

    sec_a = torch.cat([gu_tiles(cg), gu_tiles(cu), gu_scales(bg), gu_scales(bu)], dim=1).reshape(-1)
    ar = lambda n: torch.arange(n, device=dev)
    cb, ng, uu, w, g, q, j, e = torch.meshgrid(ar(CB), ar(NG), ar(8), ar(nwd), ar(8), ar(4), ar(4), ar(8), indexing="ij")
    t = cd[128 * ng + 16 * uu + 4 * q + e // 2, cb * cbw + (4 * w + j) * 16 + g + 8 * (e & 1)]
    sec_b = (t[..., 0::2] | (t[..., 1::2] << 4)).reshape(-1)
    ng2, cb2, w2, g2, j2, half, m = torch.meshgrid(ar(NG), ar(CB), ar(nwd), ar(8), ar(4), ar(2), ar(4), indexing="ij")
    sec_c = bd[4 * ng2 + m, cb2 * cbw + (4 * w2 + j2) * 16 + g2 + 8 * half].reshape(-1)
    return torch.cat([sec_a, sec_b, sec_c])


def _pack_mxfp4tc_record(cg, cu, cd, bg, bu, bd) -> torch.Tensor:
    """The inputs of ``_pack_mxfp4_record`` -> the record of operand images (see the module text), uint8 flat."""
    I, d = cg.shape
    NG, KS = I // 128, d // 128

    def images(c, R, Kd):      # codes [R rows][Kd] -> [R/128][Kd/128][8192]
        t = c.reshape(R // 128, 16, 8, Kd // 128, 2, 2, 16, 2)        # rg, r8, r, st, step, kcore, byte, nibble
        t = t.permute(0, 3, 4, 5, 1, 2, 6, 7)                          # rg, st, step, kcore, r8, r, byte, nibble
        return (t[..., 0] | (t[..., 1] << 4)).reshape(R // 128, Kd // 128, 8192)

    def scales(b_, R, Kd):     # scale bytes [R][Kd/32] -> [R/128][Kd/128][512]: (r%32)*16 + (r//32)*4 + b
        t = b_.reshape(R // 128, 4, 32, Kd // 128, 4)                  # rg, r//32, r%32, st, b
        return t.permute(0, 3, 2, 1, 4).reshape(R // 128, Kd // 128, 512)

    sec_a = torch.cat([images(cg, I, d), images(cu, I, d), scales(bg, I, d), scales(bu, I, d)], dim=2).reshape(-1)
    # down: rows are output columns, the contraction index is the neuron
    sec_b = torch.cat([images(cd.t().contiguous(), d, I), scales(bd.t().contiguous(), d, I)], dim=2).reshape(-1)
    return torch.cat([sec_a, sec_b])


def _e2m1_codes(v: torch.Tensor) -> torch.Tensor:
    """Scaled values -> e2m1 codes (uint8 0..15): nearest magnitude, ties to the even code, saturating at 6."""
    a = v.abs().clamp(max=6.0)
    bounds = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], device=v.device, dtype=torch.float32)
    lo_ = torch.bucketize(a, bounds, right=False)
    hi_ = torch.bucketize(a, bounds, right=True)
    idx = torch.where(lo_ != hi_, torch.where(lo_ % 2 == 0, lo_, hi_), lo_)
    return (idx | torch.where(v < 0, 8, 0)).to(torch.uint8)


def _quantise_nvfp4(w: torch.Tensor, block_axis: int) -> tuple[torch.Tensor, torch.Tensor, float]:
    """Two-level FP4 quantiser used to *produce* the synthetic pool: blocks of 16 along ``block_axis``.

    Matrix scale = amax / (6 * 448) (the largest block scale is the largest e4m3 number); block scale = block amax /
    (6 * matrix scale) rounded to e4m3; elements rounded to the nearest e2m1 value of w / (block scale * matrix
    scale).  Returns (codes uint8 with w's shape, scale bytes uint8 with the block axis reduced by 16, matrix scale).
    """
    I, d = w.shape
    wb = w.reshape(I, d // NV_BLOCK, NV_BLOCK) if block_axis == 1 else w.reshape(I // NV_BLOCK, NV_BLOCK, d)
    ax = 2 if block_axis == 1 else 1
    top = w.abs().max().to(torch.float32)
    ms = torch.where(top > 0, top / (6.0 * 448.0), torch.ones_like(top))
    amax = wb.abs().amax(dim=ax, keepdim=True)
    s8 = (amax / (6.0 * ms)).clamp(max=448.0).to(torch.float8_e4m3fn)
    sb = s8.to(torch.float32)
    v = torch.where(sb > 0, wb / (torch.where(sb > 0, sb, torch.ones_like(sb)) * ms), torch.zeros_like(wb))
    return _e2m1_codes(v).reshape(I, d), s8.view(torch.uint8).squeeze(ax), float(ms)


def _pack_nvfp4_record(cg, cu, cd, bg, bu, bd, scales) -> torch.Tensor:
    """Codes uint8 ``[I][d]`` (gate/up: one row per neuron; down: ``[n][c]``), scale bytes ``bg, bu [I][d/16]``,
    ``bd [I/16][d]``, the three matrix scales -> the tiled record, uint8 flat."""
    I, d = cg.shape
    dev = cg.device
    U, G, NG = I // 16, d // GROUP, I // GROUP
    nwd = min(16, d // 64)
    cbw = 64 * nwd
    CB = d // cbw

    def gu_tiles(c):      # [U][16 rows][G][j][half][q][r] -> [U][G][row][q][j][r][half], nibble e = 2 r + half
        t = c.reshape(U, 16, G, 4, 2, 4, 4).permute(0, 2, 1, 5, 3, 6, 4)
        return (t[..., 0] | (t[..., 1] << 4)).reshape(U, G * 1024)

    def gu_scales(b_):    # [U][half][r][G][k] -> [U][G][r][half][k]
        return b_.reshape(U, 2, 8, G, 8).permute(0, 3, 2, 1, 4).reshape(U, G * 128)

    sec_a = torch.cat([gu_tiles(cg), gu_tiles(cu), gu_scales(bg), gu_scales(bu)], dim=1).reshape(-1)
    ar = lambda n: torch.arange(n, device=dev)
    cb, ng, uu, w, g, q, j, e = torch.meshgrid(ar(CB), ar(NG), ar(8), ar(nwd), ar(8), ar(4), ar(4), ar(8), indexing="ij")
    t = cd[128 * ng + 16 * uu + 4 * q + e // 2, cb * cbw + (4 * w + j) * 16 + g + 8 * (e & 1)]
    sec_b = (t[..., 0::2] | (t[..., 1::2] << 4)).reshape(-1)
    ng2, cb2, w2, g2, j2, half, m = torch.meshgrid(ar(NG), ar(CB), ar(nwd), ar(8), ar(4), ar(2), ar(8), indexing="ij")
    sec_c = bd[8 * ng2 + m, cb2 * cbw + (4 * w2 + j2) * 16 + g2 + 8 * half].reshape(-1)
    tail = torch.zeros(NV_TAIL, dtype=torch.uint8, device=dev)
    tail[:12] = torch.tensor(scales, dtype=torch.float32).view(torch.uint8).to(dev)
    return torch.cat([sec_a, sec_b, sec_c, tail])


WD_NU = (0, 0, 1, 1, 2, 2, 3, 3)     # neuron offset (plus 4q) of nibble e in a word of the down section


def _pack_int4_record(qg, qu, qd, sg, su, sd) -> torch.Tensor:
    """Codes int8 ``[I][d]`` (gate/up: one row per neuron; down: ``[n][c]``), scales bf16 ``sg, su [I][d/128]``,
    ``sd [I/128][d]`` -> the tiled record, uint8 flat."""
    I, d = qg.shape
    dev = qg.device
    U, G, NG = I // 16, d // GROUP, I // GROUP
    nwd = min(16, d // 64)
    cbw = 64 * nwd
    CB = d // cbw

    def gu_tiles(q):      # [U][16 rows][G][j][q][e] -> [U][G][row][q][j][e], nibbles packed along e
        t = q.reshape(U, 16, G, 4, 4, 8).permute(0, 2, 1, 4, 3, 5)
        return _pack_nibbles(t).reshape(U, G * 1024)

    def gu_scales(s_):    # [U][half][r][G] -> [U][G][r][half]
        t = s_.reshape(U, 2, 8, G).permute(0, 3, 2, 1).contiguous()
        return t.view(torch.uint8).reshape(U, G * 32)

    sec_a = torch.cat([gu_tiles(qg), gu_tiles(qu), gu_scales(sg), gu_scales(su)], dim=1).reshape(-1)
    # section B: gather the code of every nibble position
    ar = lambda n: torch.arange(n, device=dev)
    cb, ng, uu, w, g, q, j, e = torch.meshgrid(ar(CB), ar(NG), ar(8), ar(nwd), ar(8), ar(4), ar(4), ar(8), indexing="ij")
    nu = torch.tensor(WD_NU, device=dev)[e]
    n_idx = 128 * ng + 16 * uu + 4 * q + nu
    c_idx = cb * cbw + (4 * w + j) * 16 + g + 8 * (e & 1)
    sec_b = _pack_nibbles(qd[n_idx, c_idx]).reshape(-1)
    ng2, cb2, w2, g2, j2, half = torch.meshgrid(ar(NG), ar(CB), ar(nwd), ar(8), ar(4), ar(2), indexing="ij")
    sec_c = sd[ng2, cb2 * cbw + (4 * w2 + j2) * 16 + g2 + 8 * half].contiguous().view(torch.uint8).reshape(-1)
    return torch.cat([sec_a, sec_b, sec_c])


def _pack_bf16_tiles(w: torch.Tensor) -> torch.Tensor:
    """bf16 ``[3][I][d]`` (gate and up one row per neuron, down ``[n][c]``) -> the tiled record, flat."""
    _, I, d = w.shape
    U = I // 16
    # gate / up: [unit][group][row][tile][chunk][element] -> [unit][tile][group][row][position][element]
    gu = w[0:2].reshape(2, U, 2, 8, d // 32, 4, 8).permute(0, 1, 4, 2, 3, 5, 6)
    row = torch.arange(8, device=w.device)
    pos = torch.arange(4, device=w.device)
    src = pos[None, :] ^ (row[:, None] >> 1)                    # chunk stored at position pos of row r
    gu = gu[:, :, :, :, row[:, None], src, :].reshape(2, U, 16 * d)
    # down: [unit][chunk][element][tile][group][row] -> [unit][tile][group][row][position][element]
    dn = w[2].reshape(U, 2, 8, d // 16, 2, 8).permute(0, 3, 4, 5, 1, 2)
    pos2 = torch.arange(2, device=w.device)
    src2 = pos2[None, :] ^ (row[:, None] >> 2)
    dn = dn[:, :, :, row[:, None], src2, :].reshape(U, 16 * d)
    return torch.cat([gu[0], gu[1], dn], dim=1).contiguous().reshape(-1)


def make_records(shape: LayerShape, seed: int, layer: int, first: int, count: int,
                 device="cpu", std: float = 0.02) -> torch.Tensor:
    """Records of experts ``first .. first+count-1`` of ``layer`` as uint8 ``[count, S]``.

    Record ``e`` depends only on (seed, layer, e) for a given device type, so a
    pool may be produced in chunks of any size.
    """
    I, d = shape.inter, shape.d
    out = torch.empty((count, shape.expert_bytes), dtype=torch.uint8, device=device)
    for j in range(count):
        g = _gen(device, mix64(seed, _TAG_W, layer, first + j))
        w = torch.randn((3, I, d), generator=g, device=device, dtype=torch.float32) * std
        if shape.wdtype == "bf16":
            out[j] = _pack_bf16_tiles(w.to(torch.bfloat16)).view(torch.uint8)
        elif shape.wdtype == "mxfp4":
            cg, bg = _quantise_mxfp4(w[0], 1)
            cu, bu = _quantise_mxfp4(w[1], 1)
            cd, bd = _quantise_mxfp4(w[2], 0)
            out[j] = _pack_mxfp4_record(cg, cu, cd, bg, bu, bd)
        elif shape.wdtype == "mxfp4tc":
            cg, bg = _quantise_mxfp4(w[0], 1)
            cu, bu = _quantise_mxfp4(w[1], 1)
            cd, bd = _quantise_mxfp4(w[2], 0)
            out[j] = _pack_mxfp4tc_record(cg, cu, cd, bg, bu, bd)
        elif shape.wdtype == "nvfp4":
            cg, bg, mg = _quantise_nvfp4(w[0], 1)
            cu, bu, mu = _quantise_nvfp4(w[1], 1)
            cd, bd, md = _quantise_nvfp4(w[2], 0)
            out[j] = _pack_nvfp4_record(cg, cu, cd, bg, bu, bd, (mg, mu, md))
        else:
            qg, sg = _quantise_int4(w[0:1], 2)
            qu, su = _quantise_int4(w[1:2], 2)
            qd, sd = _quantise_int4(w[2:3], 1)
            out[j] = _pack_int4_record(qg[0], qu[0], qd[0], sg[0], su[0], sd[0])
    return out


def fill_pool(pool: torch.Tensor, shape: LayerShape, n_layers: int, seed: int,
              device="cpu", chunk: int = 16, n_per_layer: int | None = None) -> None:
    """Write all records of ``n_layers`` layers into ``pool`` (uint8, host)."""
    S = shape.expert_bytes
    E = shape.n_experts if n_per_layer is None else n_per_layer
    assert pool.dtype == torch.uint8 and pool.numel() >= n_layers * E * S
    view = pool[: n_layers * E * S].view(n_layers * E, S)
    for l in range(n_layers):
        for first in range(0, E, chunk):
            cnt = min(chunk, E - first)
            rec = make_records(shape, seed, l, first, cnt, device=device)
            view[l * E + first: l * E + first + cnt].copy_(rec)
    if torch.device(device).type == "cuda":
        torch.cuda.synchronize()


def make_shared_records(shape: LayerShape, n_layers: int, seed: int, device="cpu") -> torch.Tensor:
    """Records of the always-resident shared expert of each layer, uint8 ``[L, S]`` (host)."""
    recs = [make_records(shape, seed, l, shape.n_experts, 1, device=device).cpu() for l in range(n_layers)]
    return torch.cat(recs, dim=0).contiguous()


# --------------------------------------------------------------------------
# router logits
# --------------------------------------------------------------------------

def zipf_bias(n_experts: int, alpha: float, seed: int, layer: int) -> np.ndarray:
    """``b_e = -alpha * ln(rank_e)``, rank a seeded permutation of 1..E (float64)."""
    rng = np.random.Generator(np.random.PCG64(mix64(seed, _TAG_RANK, layer)))
    rank = rng.permutation(n_experts) + 1
    return -alpha * np.log(rank.astype(np.float64))


def ar1_logits(n_layers: int, n_steps: int, batch: int, n_experts: int, rho: float,
               alpha: float, seed: int) -> np.ndarray:
    """Decode logits, float32 ``[n_steps, n_layers, batch, E]``.

    One chain per (layer, batch row): ``u_0 ~ N(0,1)``,
    ``u_t = rho*u_{t-1} + sqrt(1-rho^2)*eps_t``, ``z_t = u_t + b_layer``.
    """
    out = np.empty((n_steps, n_layers, batch, n_experts), dtype=np.float32)
    s = math.sqrt(max(0.0, 1.0 - rho * rho))
    for l in range(n_layers):
        b = zipf_bias(n_experts, alpha, seed, l)
        rng = np.random.Generator(np.random.PCG64(mix64(seed, _TAG_U0, l, batch)))
        u = rng.standard_normal((batch, n_experts))
        for t in range(n_steps):
            if t > 0:
                u = rho * u + s * rng.standard_normal((batch, n_experts))
            out[t, l] = (u + b).astype(np.float32)
    return out


def prefill_logits(n_layers: int, n_tokens: int, n_experts: int, alpha: float, seed: int,
                   step: int = 0) -> np.ndarray:
    """Prefill logits ``eps + b``, float32 ``[n_layers, T, E]``."""
    out = np.empty((n_layers, n_tokens, n_experts), dtype=np.float32)
    for l in range(n_layers):
        b = zipf_bias(n_experts, alpha, seed, l)
        rng = np.random.Generator(np.random.PCG64(mix64(seed, _TAG_LOGIT, l, step)))
        out[l] = (rng.standard_normal((n_tokens, n_experts)) + b).astype(np.float32)
    return out


def normal_logits(n_tokens: int, n_experts: int, seed: int, step: int) -> np.ndarray:
    """Fresh ``N(0,1)`` logits per step (the tiny configuration), float32 ``[T, E]``."""
    rng = np.random.Generator(np.random.PCG64(mix64(seed, _TAG_LOGIT, 0, step)))
    return rng.standard_normal((n_tokens, n_experts)).astype(np.float32)


# --------------------------------------------------------------------------
# activations
# --------------------------------------------------------------------------

def noise_x(n_tokens: int, d: int, seed: int, step: int, layer: int, device="cpu") -> torch.Tensor:
    """``N(0,1)`` noise rows as bf16 ``[T, d]``; the layer input is this noise plus
    (for layer > 0) the previous layer's output, rounded to bf16 by the caller."""
    g = _gen(device, mix64(seed, _TAG_X, step, layer))
    return torch.randn((n_tokens, d), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
