"""Parity at full size, in the launch configuration the benchmark times: the whole
mistral-7B-shaped model (7.24e9 weights) compressed on the device and decoded by ONE batched
call with the default launch shape.

The oracle cannot decode 7e9 symbols bit by bit in a test, so two checks are combined:
 - a property that holds at any size, on every tensor: decoding returns the symbols that
   were encoded, dequantised by the definition out = fp16(fp32(s) * fp32(q - z)) - written
   here with plain torch operations, one fp32 product and one rounding, tolerance 0;
 - sampled tensors (small, medium and the largest matrix shape, and a norm-gain vector)
   are compressed by the CPU oracle from the same fp16 bytes, and the oracle's symbols,
   parameters, stream and dequantised output are compared element by element, tolerance 0.
"""
import numpy as np
import pytest
import torch

import bench
import oracle
import paper_2505_02380_b200 as E
import workloads
from helpers import expected_out

pytestmark = pytest.mark.gpu


def _check_model(wl, sample_names):
    E.entro_set_decode_config(*E.DEFAULT_DECODE_CONFIG)
    model = bench.DeviceModel(wl, E, E.DEFAULT_DECODE_CONFIG[0], keep_q=True)
    model.out.zero_()
    E.entro_decode_dequant_batched(model.descs)
    torch.cuda.synchronize()
    assert E.entro_last_device_status() == E.OK
    # every tensor: the definition, in torch
    for spec, q, (s, z), out in zip(wl.tensors, model.q, model.qparams, model.out_slices):
        want = (torch.tensor(s, dtype=torch.float32, device="cuda") * (q.to(torch.int32) - z).to(torch.float32))
        assert torch.equal(out.view(torch.int16), want.to(torch.float16).view(torch.int16)), spec.name
    # sampled tensors: the oracle, from the same bytes
    by_name = {t.name: i for i, t in enumerate(wl.tensors)}
    for name in sample_names:
        i = by_name[name]
        spec = wl.tensors[i]
        w = workloads.make_tensor(spec, "cuda").view(-1).cpu().numpy()
        c = oracle.compress(w, wl.bits, wl.chunk_symbols)
        s, z = model.qparams[i]
        assert (np.float32(s).tobytes(), z) == (np.float32(c.qp.scale).tobytes(), c.qp.zero_point), name
        assert torch.equal(model.q[i].cpu(), torch.from_numpy(c.q)), name
        assert torch.equal(model.keep[i].stream.cpu(), torch.from_numpy(c.enc.stream.view(np.int32))), name
        got = model.out_slices[i].cpu().numpy().view(np.uint16)
        assert np.array_equal(got, expected_out(c)), name


def test_mistral_shaped_full_model_uint8():
    _check_model(workloads.mistral_7b(bits=8),
                 ["layers.0.k_proj", "layers.17.q_proj", "layers.31.down_proj", "layers.9.input_norm"])


def test_mistral_shaped_full_model_uint4():
    _check_model(workloads.mistral_7b(bits=4),
                 ["layers.3.v_proj", "layers.20.o_proj", "layers.12.gate_proj", "final_norm"])


def test_smollm_shaped_full_model_uint8():
    """Config 2: 169 matrices + norm gains, unsigned or asymmetric per tensor by the mixed rule."""
    wl = workloads.smollm_1p7b()
    _check_model(wl, ["layers.5.k_proj", "layers.23.down_proj", "layers.11.post_attn_norm", "embed_tokens"])


def test_phi3_shaped_full_model_uint4():
    """Config 3: fused qkv / gate_up shapes, 4-bit symbols, 8192-symbol chunks."""
    _check_model(workloads.phi3_mini_4k(), ["layers.0.qkv_proj", "layers.31.down_proj", "layers.16.o_proj", "final_norm"])
