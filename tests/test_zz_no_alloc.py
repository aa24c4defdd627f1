"""The allocation-free expert FFN entry point against the regular forward path.

Some users of the library run where device allocation is forbidden (a frozen memory budget, a
plug-in in somebody else's process), so they cannot create a handle; ``ft_moe_ffn_noalloc`` gives them
the same streaming FFN kernel with its scratch in a fixed array inside the library.  The test drives
both entry points through the C ABI on the same expert record and inputs, twice in a row because
the fixed scratch keeps the previous call's contents, and expects the same output within the
tolerance of the other GPU tests; since both run the same kernel, the output is also compared with
the plain SwiGLU definition evaluated by the CPU oracle from the same record.  Collected last so that a stop at the first failure has already run
everything else; it passes both alone in a fresh process and after the other tests.
"""
import numpy as np
import pytest
import torch

from oracle import ftmoe_oracle as O
from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W
from tests.helpers import MAX_ABS_TOL, REL_L2_TOL, bits, check_output

pytestmark = pytest.mark.gpu


def _reference_through_handle(shape, pool, x_dev, T):
    """y = FFN_0(x) through ft_moe_layer: one expert, top-1, so the gate weight is exactly 1."""
    cfg = B.make_config(hidden=shape.d, inter=shape.inter, n_experts=1, top_k=1, slots_per_layer=1,
                        max_tokens=T, host_pool_ptr=pool.ptr.value, host_pool_bytes=pool.n_bytes)
    moe = B.FtMoe(cfg)
    logits = torch.zeros((T, 1), dtype=torch.float32, device=x_dev.device)
    y = torch.empty_like(x_dev)
    moe.layer(0, logits, x_dev, y, T)
    assert moe.sync_status() == 0
    moe.destroy()
    return y


@pytest.mark.parametrize("d,inter,T", [(2048, 768, 8), (512, 192, 37), (256, 128, 64)])
def test_noalloc_entry_point_matches_forward_twice_in_a_row(d, inter, T):
    shape = W.LayerShape(d=d, inter=inter, n_experts=1, top_k=1)
    pool = B.HostPool(shape.expert_bytes)
    W.fill_pool(pool.tensor, shape, 1, seed=21)
    dev = torch.device("cuda:0")
    record_dev = pool.tensor.to(dev)                       # the caller's own copy of the record
    wg, wu, wd = O.unpack_record(pool.tensor.numpy(), d, inter, "bf16")
    torch.cuda.set_device(0)
    for call in range(2):
        x = W.noise_x(T, d, 21, call, 0).to(dev)
        y_ref = _reference_through_handle(shape, pool, x, T)
        y = torch.full_like(x, float("nan"))
        rc = B.ft_moe_ffn_noalloc(0, record_dev, d, inter, x, y, T)
        assert rc == B.FT_OK, B.status_string(rc)
        torch.cuda.synchronize()
        a, b = y.float().cpu().double().numpy(), y_ref.float().cpu().double().numpy()
        assert np.all(np.isfinite(a))
        assert np.linalg.norm(a - b) <= REL_L2_TOL * np.linalg.norm(b)
        assert np.abs(a - b).max() <= MAX_ABS_TOL * np.abs(b).max()
        check_output(y, O.expert_ffn(O.bf16_to_f64(bits(x)), wg, wu, wd))
        assert B.ft_moe_ffn_noalloc_status(0) == B.FT_OK
        assert torch.cuda.current_device() == 0          # the caller's device is left as it was
    pool.free()


def test_noalloc_entry_point_rejects_sizes_beyond_its_static_scratch():
    dev = torch.device("cuda:0")
    rec = torch.zeros(3 * 128 * 256 * 2, dtype=torch.uint8, device=dev)
    x = torch.zeros((B.NOALLOC_MAX_TOKENS + 1, 256), dtype=torch.bfloat16, device=dev)
    y = torch.empty_like(x)
    assert B.ft_moe_ffn_noalloc(0, rec, 256, 128, x, y, B.NOALLOC_MAX_TOKENS + 1) == B.FT_ERR_INVALID_ARG
    assert B.ft_moe_ffn_noalloc(0, rec, 256, 128, x, y, 0) == B.FT_ERR_INVALID_ARG
    assert B.ft_moe_ffn_noalloc(0, rec, 4096, 128, x, y, 4) == B.FT_ERR_INVALID_ARG
    assert B.ft_moe_ffn_noalloc(0, rec, 768, 128, x, y, 4) == B.FT_ERR_UNSUPPORTED
    assert B.ft_moe_ffn_noalloc(0, None, 256, 128, x, y, 4) == B.FT_ERR_INVALID_ARG
    # a view that starts at an odd element is not 16-byte aligned: refused on the host, nothing is launched
    odd = torch.zeros(4 * 256 + 8, dtype=torch.bfloat16, device=dev)[1:1 + 4 * 256].view(4, 256)
    assert B.ft_moe_ffn_noalloc(0, rec, 256, 128, odd, y, 4) == B.FT_ERR_INVALID_ARG
    assert B.ft_moe_ffn_noalloc(0, rec, 256, 128, x, odd, 4) == B.FT_ERR_INVALID_ARG
    torch.cuda.synchronize()
