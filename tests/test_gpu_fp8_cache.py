"""GPU parity of the FP8 K/V cache variant: against the oracle attention over the oracle's
dequantised cache, and bit for bit against tsd_verify_attention on that same dequantised cache."""
import numpy as np
import pytest
import torch

import oracle
from oracle import fp8
from paper_2608_27514_b200 import binding as B
from paper_2608_27514_b200 import workloads as W
from paper_2608_27514_b200.step import VerifyStep
from test_gpu_parity import PATHS, _attn_tol, _np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _quantise(t, scale):
    """bf16 cache [S,Nc,H,d], scale [S,H] -> e4m3 codes as uint8 (torch's conversion: a library routine)."""
    x = (t.float() / scale[:, None, :, None]).clamp(-448.0, 448.0)      # the cast does not saturate
    return x.to(torch.float8_e4m3fn).view(torch.uint8).contiguous()


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("shape", [dict(S=2, B=5, R=32, Nc=300, Hq=4, Hkv=2), dict(S=1, B=8, R=32, Nc=736, Hq=4, Hkv=4),
                                   dict(S=3, B=2, R=64, Nc=64, Hq=2, Hkv=1), dict(S=1, B=3, R=32, Nc=0, Hq=2, Hkv=2)])
def test_fp8_cache_attention(flags, shape):
    cfg = W.small(W.CONFIGS["cfg2"], **shape)
    attn = W.attention_inputs(cfg, DEV)
    step = VerifyStep.for_config(cfg, DEV)
    cache_lens = None
    if cfg.Nc > 64:
        cache_lens = torch.tensor([cfg.Nc - 37 * (s + 1) for s in range(cfg.S)], dtype=torch.int32, device=DEV)
    step.build_mask(None, cache_lens)
    g = torch.Generator(device="cpu").manual_seed(5)
    ksc = (0.5 + torch.rand((cfg.S, cfg.Hkv), generator=g)).to(DEV) / 64.0
    vsc = (0.5 + torch.rand((cfg.S, cfg.Hkv), generator=g)).to(DEV) / 64.0
    kq, vq = _quantise(attn["k_cache"], ksc), _quantise(attn["v_cache"], vsc)
    if cache_lens is not None:
        # the unused capacity holds the two NaN codes of e4m3: it is never decoded into the result
        for s_, n in enumerate(cache_lens.tolist()):
            kq[s_, n:] = 0x7F
            vq[s_, n:] = 0xFF
    ws = torch.empty(max(B.tsd_verify_attention_fp8_cache_workspace_bytes(step.layout), 16), dtype=torch.uint8, device=DEV)
    out = torch.full_like(step.out, 3.0)
    lse = torch.empty_like(step.attn_lse)
    B.tsd_verify_attention_fp8_cache(step.layout, step.mask, attn["q"], kq if cfg.Nc else None, vq if cfg.Nc else None,
                                     ksc, vsc, attn["k_draft"], attn["v_draft"], out, ws, lse, attn["sm_scale"], flags,
                                     step.status)
    torch.cuda.synchronize()
    step.check_status()
    # the cache the kernel is defined to see, from the oracle
    kd = fp8.dequant_cache(kq.cpu().numpy(), ksc.cpu().numpy())
    vd = fp8.dequant_cache(vq.cpu().numpy(), vsc.cpu().numpy())
    mask = oracle.dense_mask(cfg.S, cfg.B, cfg.R, cfg.Nc, None, None if cache_lens is None else cache_lens.cpu().numpy())
    ref, ref_lse = oracle.masked_attention(_np(attn["q"]), kd, vd, _np(attn["k_draft"]), _np(attn["v_draft"]), mask,
                                           attn["sm_scale"])
    got = _np(out).astype(np.float64)
    assert (np.abs(got - ref) <= _attn_tol(cfg, ref)).all()
    assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 2e-2
    # and bit for bit what the plain entry point gives on that dequantised cache
    if cfg.Nc:
        step.attention(attn["q"], torch.from_numpy(kd).to(DEV).bfloat16(), torch.from_numpy(vd).to(DEV).bfloat16(),
                       attn["k_draft"], attn["v_draft"], attn["sm_scale"], flags)
        torch.cuda.synchronize()
        assert torch.equal(step.out, out) and torch.equal(step.attn_lse, lse)


def test_fp8_cache_argument_checks():
    cfg = W.small(W.CONFIGS["cfg2"], S=1, B=2, R=32, Nc=64, Hq=2, Hkv=2)
    attn = W.attention_inputs(cfg, DEV)
    step = VerifyStep.for_config(cfg, DEV)
    step.build_mask()
    kq = torch.zeros((1, 64, 2, 128), dtype=torch.uint8, device=DEV)
    small = torch.empty(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.TsdError) as ei:
        B.tsd_verify_attention_fp8_cache(step.layout, step.mask, attn["q"], kq, kq, None, None, attn["k_draft"],
                                         attn["v_draft"], step.out, small)
    assert ei.value.code == B.TSD_ERR_WORKSPACE
    f32 = W.small(W.CONFIGS["cfg1"], S=1, B=2, R=32, Nc=64, Hq=2, Hkv=2)
    lay = B.make_layout(1, 2, 32, 64, 2, 2, 64, torch.float32)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.TsdError) as ei:
        B.tsd_verify_attention_fp8_cache(lay, step.mask, attn["q"], kq, kq, None, None, attn["k_draft"],
                                         attn["v_draft"], step.out, ws)
    assert ei.value.code == B.TSD_ERR_UNSUPPORTED
