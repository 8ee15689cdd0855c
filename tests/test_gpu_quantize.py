"""GPU parity of the 8-bit codes of retained values against the CPU oracle: codes and scale bit for bit, decoded
values bit for bit, and the weight gradient from a quantised cache against Eq. 6 on the oracle's decoded values."""
import numpy as np
import pytest
import torch

import dropit_inputs as di
import oracle
import paper_2202_13808_b200 as dropit
from _parity import max_rel_err, np_bits, oracle_cache

pytestmark = pytest.mark.gpu


def _roundtrip(bits_np, dev):
    """Quantise an arbitrary array of bf16 patterns on the GPU through a cache object."""
    vals = torch.from_numpy(bits_np.view(np.int16).copy()).view(torch.bfloat16).to(dev)
    n = vals.numel()
    cache = dropit.DropITCache(vals, torch.empty(0, dtype=torch.int32, device=dev),
                               torch.zeros(1, dtype=torch.int32, device=dev), n, n, (n,), torch.bfloat16, 0, 0.0)
    q = dropit.dropit_quantize_cache(cache)
    back = dropit.dropit_dequantize_cache(q)
    return q.codes.cpu().numpy(), int(q.scale.item()), np_bits(back.values)


def test_every_bf16_pattern_under_several_scales(cuda_device):
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    for top in (0x3F80, 0x4100, 0x7F00, 0x0600, 0x0500):             # the largest finite value fixes the scale
        keyv = allbits & 0x7FFF
        sel = allbits[(keyv <= top) | (keyv >= 0x7F80)]               # everything up to the top value, plus Inf / NaN
        codes, e_top, dec = _roundtrip(sel, cuda_device)
        assert e_top == oracle.q8_top_exponent(sel) == (top >> 7)
        exp_codes = oracle.q8_encode(sel, e_top)
        assert (codes == exp_codes).all()
        assert (dec == oracle.q8_decode(exp_codes, e_top)).all()


@pytest.mark.parametrize("case", [di.small_linear(640, 768, 384, "bf16", 0.9), di.small_linear(300, 3072, 128, "bf16", 0.9, "gelu"),
                                  di.VITB_FC1], ids=lambda c: c.name)
def test_weight_grad_from_a_quantised_cache(cuda_device, case):
    x, dy = di.make_x(case), di.make_dy(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    dyb, _ = oracle.to_bits(dy)
    cache = dropit.dropit_compress(x.to(cuda_device), case.gamma, "bitmask")
    q = dropit.dropit_quantize_cache(cache)
    vals = oracle.pack_values(bits, keep, dt)
    e_top = oracle.q8_top_exponent(vals)
    codes = oracle.q8_encode(vals, e_top)
    assert int(q.scale.item()) == e_top and (q.codes.cpu().numpy() == codes).all()
    assert q.nbytes < cache.nbytes - k + 8 and q.values is None
    # the oracle's Eq. 6 on the tensor whose retained entries are the decoded codes
    xq = bits.copy()
    xq[keep == 1] = oracle.q8_decode(codes, e_top)
    dw = dropit.dropit_weight_grad(dy.to(cuda_device), q)
    dropit.check_device_status(cuda_device)
    if case.n <= 2_000_000:
        ref = oracle.fc_weight_grad(dyb, xq, keep, case.M, case.Ca, case.Cz, dt)
        assert max_rel_err(dw.cpu().numpy(), ref) <= 2e-4
        exact = oracle.fc_weight_grad(dyb, bits, keep, case.M, case.Ca, case.Cz, dt)
        assert max_rel_err(dw.cpu().numpy(), exact) <= 3e-2      # 1 part in 32 per value, averaged over the sum
    else:
        rng = np.random.default_rng(0)
        js, cs = rng.integers(0, case.Cz, 1500), rng.integers(0, case.Ca, 1500)
        ref = oracle.fc_weight_grad_entries(dyb, xq, keep, case.M, case.Ca, case.Cz, dt, js, cs)
        assert np.abs(dw.cpu().numpy()[js, cs] - ref).max() / np.abs(ref).max() <= 2e-4


def test_linear_layer_with_quantised_cache(cuda_device):
    from paper_2202_13808_b200.nn import DropITLinear
    torch.manual_seed(0)
    lin = DropITLinear(768, 384, gamma=0.9, quantize=True, device=cuda_device, dtype=torch.bfloat16).train()
    ref = DropITLinear(768, 384, gamma=0.9, device=cuda_device, dtype=torch.bfloat16).train()
    ref.weight.data.copy_(lin.weight.data); ref.bias.data.copy_(lin.bias.data)
    x = torch.randn(4096, 768, device=cuda_device, dtype=torch.bfloat16, requires_grad=True)
    dz = (torch.randn(4096, 384, device=cuda_device) * 0.02).to(torch.bfloat16)
    z = lin(x)
    saved = [t for t in z.grad_fn.saved_tensors if t.data_ptr() != lin.weight.data_ptr()]
    z.backward(dz)
    ref(x.detach()).backward(dz)
    kept = dropit.dropit_keep_count(x.numel(), 0.9)
    assert any(t.dtype == torch.uint8 and t.numel() == kept for t in saved)          # one byte per retained value
    assert sum(t.numel() * t.element_size() for t in saved) < 0.14 * x.numel() * 2     # 5 + 6.25 + 1.6 % of the dense tensor
    err = (lin.weight.grad.float() - ref.weight.grad.float()).abs().max() / ref.weight.grad.float().abs().max()
    assert float(err) < 3e-2
    dropit.check_device_status(cuda_device)
