"""The allocation-free layer entry point (pd_encoder_layer_fwd_static).

Some users of the library cannot allocate device memory where they call it (a
server whose pool owns the GPU, a plug-in without an allocator, a place where
cudaMalloc's device-wide synchronisation is unacceptable).  For them the layer
keeps its intermediates in a fixed array inside the library.  This test calls
that entry point through the C ABI twice in a row and checks both results
against the ordinary entry point (and, on the smaller shape, against the CPU
oracle directly).  The file sorts last on purpose.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_03586_b200 import inputs
from parity import dev_bf16, dev_f32, host, max_rel_floored

pytestmark = pytest.mark.gpu
TOL = 2e-2

_MATS = ("w_qkv", "w_o", "w_ffn1", "w_ffn2")
_VECS = ("b_qkv", "b_o", "b_ffn1", "b_ffn2", "ln1_gamma", "ln1_beta", "ln2_gamma", "ln2_beta")


def _setup(api, shape, seed, want_inputs=False):
    p = inputs.encoder_layer_inputs(shape, seed=seed)
    kw = {m: dev_bf16(p[m + "_bits"]) for m in _MATS}
    kw.update({v: dev_f32(p[v]) for v in _VECS})
    out = api.EncoderLayerParams(**kw), dev_bf16(p["x_bits"])
    return out + (p,) if want_inputs else out


def _oracle_layer(p, shape):
    w = {m: inputs.bf16_bits_to_f32(p[m + "_bits"]) for m in _MATS}
    return oracle.encoder_layer(inputs.bf16_bits_to_f32(p["x_bits"]), w["w_qkv"], p["b_qkv"], w["w_o"], p["b_o"],
                                w["w_ffn1"], p["b_ffn1"], w["w_ffn2"], p["b_ffn2"], p["ln1_gamma"], p["ln1_beta"],
                                p["ln2_gamma"], p["ln2_beta"], batch=shape.batch, seq=shape.seq, heads=shape.heads,
                                ln_eps=np.float32(shape.ln_eps))


def test_static_scratch_layer_matches_workspace_layer_twice():
    from paper_2511_03586_b200 import api
    api.pd_clear_device_status()
    assert api.pd_encoder_layer_static_scratch_bytes() == 32 << 20
    # two different problems back to back: the second call finds the first one's leftovers in the array
    for shape, seed in ((inputs.EncoderLayerShape(batch=2, seq=384, hidden=256, heads=4, ffn=1024), 1),
                        (inputs.EncoderLayerShape(batch=1, seq=512, hidden=1024, heads=16, ffn=4096), 2)):
        params, x, p = _setup(api, shape, seed, want_inputs=True)
        kw = dict(batch=shape.batch, seq=shape.seq, heads=shape.heads)
        expect = api.pd_encoder_layer_fwd(params, x, **kw)
        ref = _oracle_layer(p, shape) if shape.hidden == 256 else None   # the small shape: a few seconds of oracle time
        assert api.pd_encoder_layer_workspace_bytes(shape.batch, shape.seq, shape.hidden, shape.heads, shape.ffn) \
            <= api.pd_encoder_layer_static_scratch_bytes()
        y = torch.full_like(x, float("nan"))
        for _ in range(2):
            api.pd_encoder_layer_fwd_static(params, x, y, **kw)
            torch.cuda.synchronize()
            assert max_rel_floored(host(y), host(expect)) < TOL
            assert torch.equal(y, expect)          # same kernels, same order: in fact bit-identical
            if ref is not None:
                assert max_rel_floored(host(y), ref) < TOL
            y.fill_(float("nan"))
    assert api.pd_get_device_status() == 0


def test_static_scratch_layer_rejects_oversized_shapes():
    from paper_2511_03586_b200 import api
    shape = inputs.EncoderLayerShape(batch=4, seq=512, hidden=1024, heads=16, ffn=4096)   # needs ~44 MiB
    assert api.pd_encoder_layer_workspace_bytes(4, 512, 1024, 16, 4096) > api.pd_encoder_layer_static_scratch_bytes()
    params, x = _setup(api, shape, 3)
    y = torch.zeros_like(x)
    with pytest.raises(api.PdError, match="PD_ERR_WORKSPACE_TOO_SMALL"):
        api.pd_encoder_layer_fwd_static(params, x, y, batch=4, seq=512, heads=16)
    assert not bool(y.any())                      # nothing was enqueued
