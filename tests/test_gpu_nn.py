"""GPU tests of the autograd wrappers (Sec. 3.2 / 3.5, Fig. 1b, App. A.6): gradients, saved tensors, memory."""
import numpy as np
import pytest
import torch
import torch.nn as nn
import torch.nn.functional as F

import dropit_inputs as di
import oracle
import paper_2202_13808_b200 as dropit
from paper_2202_13808_b200.nn import DropITConv2d, DropITLinear, convert_linear_layers
from _parity import max_rel_err, oracle_cache

pytestmark = pytest.mark.gpu


def test_linear_wrapper_gradients(cuda_device):
    case = di.small_linear(640, 768, 384, "bf16", 0.9)
    x = di.make_x(case).to(cuda_device).reshape(5, 128, 768).requires_grad_(True)
    dy = di.make_dy(case).to(cuda_device).reshape(5, 128, 384)
    torch.manual_seed(0)
    lin = DropITLinear(768, 384, gamma=0.9, device=cuda_device, dtype=torch.bfloat16).train()
    ref = nn.Linear(768, 384, device=cuda_device, dtype=torch.bfloat16)
    ref.weight.data.copy_(lin.weight.data); ref.bias.data.copy_(lin.bias.data)
    z = lin(x)
    z.backward(dy)
    x2 = x.detach().clone().requires_grad_(True)
    z2 = ref(x2)
    z2.backward(dy)
    # forward, input gradient (Eq. 3) and bias gradient are untouched by DropIT
    assert torch.equal(z, z2) and torch.equal(x.grad, x2.grad)
    assert torch.allclose(lin.bias.grad.float(), ref.bias.grad.float(), rtol=2e-2, atol=1e-3)
    # the weight gradient is the oracle's Eq. 6 on the compressed cache, rounded to the parameter dtype
    bits, dt, keep, k = oracle_cache(x.detach().cpu().reshape(-1, 768), 0.9)
    dyb, _ = oracle.to_bits(dy.cpu().reshape(-1, 384))
    dw = oracle.fc_weight_grad(dyb, bits, keep, 640, 768, 384, dt)
    assert max_rel_err(lin.weight.grad.float().cpu().numpy(), dw) < 1e-2
    dropit.check_device_status(cuda_device)


def test_linear_wrapper_gamma_zero_equals_stock(cuda_device):
    torch.manual_seed(1)
    lin = DropITLinear(256, 128, gamma=0.0, device=cuda_device, dtype=torch.float32).train()
    x = torch.randn(300, 256, device=cuda_device, requires_grad=True)
    dy = torch.randn(300, 128, device=cuda_device)
    lin(x).backward(dy)
    ref = dy.double().t() @ x.detach().double()
    assert max_rel_err(lin.weight.grad.cpu().numpy(), ref.cpu().numpy()) < 1e-5


def test_conv_wrapper_gradients(cuda_device):
    case = di.small_conv(2, 16, 14, 14, 32, 3, 3, 1, 1, "bf16", 0.8)
    x = di.make_x(case).to(cuda_device).requires_grad_(True)
    dy = di.make_dy(case).to(cuda_device)
    torch.manual_seed(2)
    conv = DropITConv2d(16, 32, 3, padding=1, gamma=0.8, device=cuda_device, dtype=torch.bfloat16).train()
    z = conv(x)
    z.backward(dy)
    z2 = F.conv2d(x.detach(), conv.weight, conv.bias, 1, 1)
    assert torch.equal(z, z2)
    dx_ref = torch.nn.grad.conv2d_input(x.shape, conv.weight, dy, stride=1, padding=1)
    assert torch.equal(x.grad, dx_ref)
    bits, dt, keep, k = oracle_cache(x.detach().cpu(), 0.8)
    dyb, _ = oracle.to_bits(dy.cpu())
    dw = oracle.conv_weight_grad(dyb, bits, keep, 2, 16, 14, 14, 32, 3, 3, 1, 1, dt)
    assert max_rel_err(conv.weight.grad.float().cpu().numpy(), dw) < 1e-2


def test_only_the_compressed_cache_is_saved(cuda_device):
    lin = DropITLinear(768, 768, gamma=0.9, device=cuda_device, dtype=torch.bfloat16).train()
    x = torch.randn(4096, 768, device=cuda_device, dtype=torch.bfloat16, requires_grad=True)
    z = lin(x)
    saved = z.grad_fn.saved_tensors
    dense_bytes = x.numel() * 2
    saved_bytes = sum(t.numel() * t.element_size() for t in saved if t.data_ptr() != lin.weight.data_ptr())
    assert all(t.data_ptr() != x.data_ptr() for t in saved)
    assert saved_bytes < 0.19 * dense_bytes       # 10% values + 6.25% mask + 1.6% table


def test_eval_mode_is_the_stock_layer(cuda_device):
    lin = DropITLinear(64, 32, device=cuda_device, dtype=torch.float32).eval()
    x = torch.randn(8, 64, device=cuda_device)
    assert torch.equal(lin(x), F.linear(x, lin.weight, lin.bias))


def test_activation_memory_shrinks_with_dropit(cuda_device):
    """A stack of Linear+GELU.  GELU caches its own input (kept dense, Sec. 3.5) but not its output, so the
    Linear inputs are held by the Linear layers alone and DropIT at gamma=0.9 must lower the peak.  (With
    ReLU, which caches its output, the dense tensor stays alive and DropIT cannot save anything.)"""
    def peak(gamma):
        torch.manual_seed(3)
        layers = []
        for _ in range(6):
            layers += [nn.Linear(1024, 1024), nn.GELU()]
        model = nn.Sequential(*layers).to(cuda_device, torch.bfloat16).train()
        if gamma is not None:
            convert_linear_layers(model, gamma)
        x = torch.randn(16384, 1024, device=cuda_device, dtype=torch.bfloat16)
        for _ in range(2):
            model.zero_grad(set_to_none=True)
            torch.cuda.synchronize()
            base = torch.cuda.memory_allocated(cuda_device)
            torch.cuda.reset_peak_memory_stats(cuda_device)
            model(x).float().pow(2).mean().backward()
            torch.cuda.synchronize()
            p = torch.cuda.max_memory_allocated(cuda_device) - base
        return p
    dense, sparse = peak(None), peak(0.9)
    assert sparse < 0.9 * dense, (dense, sparse)   # GELU caches and backward temporaries are common to both


def test_vit_step_runs_with_dropit_on_every_linear(cuda_device):
    from paper_2202_13808_b200.vit import build_vit_b16, train_steps
    model = build_vit_b16(0.9, device=cuda_device, depth=2)
    n_dropit = sum(isinstance(m, DropITLinear) for m in model.modules())
    assert n_dropit == 2 * 4 + 1
    sps, peak, loss = train_steps(model, batch=8, steps=2, warmup=1)
    assert sps > 0 and np.isfinite(loss)
    dropit.check_device_status(cuda_device)


def test_gelu_linear_module_uses_the_producer_and_matches_the_oracle(cuda_device):
    """GELU + Linear with the GELU written by dropit_produce: the forward is the correctly rounded GELU followed by
    the stock matmul, the weight gradient is Eq. 6 on the min-k cache of GELU(x), the input gradient goes through
    the activation's own (dense) cache."""
    from paper_2202_13808_b200.nn import DropITGeluLinear
    torch.manual_seed(3)
    M, Ca, Cz = 1024, 768, 256                       # 786 432 elements: large enough for the sampled path
    x = torch.randn(M, Ca, device=cuda_device).to(torch.bfloat16).requires_grad_(True)
    dz = (torch.randn(M, Cz, device=cuda_device) * 0.02).to(torch.bfloat16)
    lin = DropITGeluLinear(Ca, Cz, gamma=0.9, device=cuda_device, dtype=torch.bfloat16).train()
    z = lin(x)
    z.backward(dz)
    # forward: table GELU (rounded once from double) then F.linear
    xb = x.detach().cpu().view(torch.int16).numpy().view(np.uint16).reshape(-1)
    yb = oracle.apply_table(oracle.activation_table(oracle.ACT_GELU), xb)
    y = torch.from_numpy(yb.view(np.int16)).view(torch.bfloat16).reshape(M, Ca).to(cuda_device)
    assert torch.equal(z, F.linear(y, lin.weight, lin.bias))
    # weight gradient: the oracle's Eq. 6 on min-k of GELU(x)
    keep, k = oracle.min_k(yb, 0.9, oracle.BF16)
    dzb, _ = oracle.to_bits(dz.cpu())
    dw = oracle.fc_weight_grad(dzb, yb, keep, M, Ca, Cz, oracle.BF16)
    assert max_rel_err(lin.weight.grad.float().cpu().numpy(), dw) < 1e-2
    # input gradient: stock GELU backward of dz W
    x2 = x.detach().clone().requires_grad_(True)
    F.linear(F.gelu(x2), lin.weight, lin.bias).backward(dz)
    assert torch.allclose(x.grad.float(), x2.grad.float(), rtol=2e-2, atol=1e-4)
    dropit.check_device_status(cuda_device)


def test_fp32_activation_in_front_of_bf16_weights_is_cached_in_bf16(cuda_device):
    """Under autocast (or with fp32 activations and bf16 weights) the matmul runs in bf16, so the cache is bf16:
    a third of the bytes of an fp32 cache, and the tensor-core weight gradient."""
    torch.manual_seed(4)
    lin = DropITLinear(256, 128, gamma=0.9, device=cuda_device, dtype=torch.float32).train()
    x = torch.randn(4096, 256, device=cuda_device, requires_grad=True)
    saved = []
    with torch.autograd.graph.saved_tensors_hooks(lambda t: (saved.append(t), t)[1], lambda t: t):
        with torch.autocast("cuda", dtype=torch.bfloat16):
            z = lin(x)
    assert z.dtype == torch.bfloat16
    assert any(t.dtype == torch.bfloat16 and t.numel() == dropit.dropit_keep_count(x.numel(), 0.9) for t in saved)
    z.float().sum().backward()
    assert lin.weight.grad is not None and torch.isfinite(lin.weight.grad).all()
    dropit.check_device_status(cuda_device)


def test_vit_step_with_the_gelu_fused_into_fc2(cuda_device):
    from paper_2202_13808_b200.nn import DropITGeluLinear
    from paper_2202_13808_b200.vit import build_vit_b16, train_steps
    model = build_vit_b16(0.9, device=cuda_device, depth=2, fuse_gelu=True)
    assert sum(isinstance(m, DropITGeluLinear) for m in model.modules()) == 2
    assert sum(isinstance(m, DropITLinear) for m in model.modules()) == 2 * 3 + 1
    sps, peak, loss = train_steps(model, batch=8, steps=2, warmup=1)
    assert sps > 0 and np.isfinite(loss)
    dropit.check_device_status(cuda_device)


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs two visible devices")
def test_second_device_in_the_same_process():
    """Kernel attributes and cached plans are kept per device: after cuda:0 has been used, cuda:1 compresses and
    takes a weight gradient in the same process (each GPU works on its own memory only; no peer access)."""
    case = di.small_linear(640, 768, 384, "bf16", 0.9)
    x, dy = di.make_x(case), di.make_dy(case)
    bits, dt, keep, k = oracle_cache(x, case.gamma)
    dyb, _ = oracle.to_bits(dy)
    ref = oracle.fc_weight_grad(dyb, bits, keep, case.M, case.Ca, case.Cz, dt)
    for dev in (torch.device("cuda:0"), torch.device("cuda:1")):
        cache = dropit.dropit_compress(x.to(dev), case.gamma, "bitmask")
        dw = dropit.dropit_weight_grad(dy.to(dev), cache)
        dwf = dropit.dropit_weight_grad(dy.to(dev), cache, fused=True)
        dropit.check_device_status(dev)
        assert cache.k == k
        assert max_rel_err(dw.cpu().numpy(), ref) < 2e-4 and max_rel_err(dwf.cpu().numpy(), ref) < 2e-4
