"""Parity at full size, in the launch configuration the benchmark times: a whole model
compressed on the device and decoded by ONE batched call with the default launch shape.

Every tensor of every model meets the oracle: its fp16 bytes are copied to the host, the
oracle quantises them (range, mode, s, z, symbols: O(n) loops) and dequantises its own
symbols, and the library's parameters, symbols and decoded fp16 output are compared with
that element by element, tolerance 0.  What decoding must return is, by the method's own
definition, the dequantised symbols, so this checks the whole decode at full size against
the oracle without the oracle having to walk 7e9 codes bit by bit.  The oracle's tensors
are independent of one another and are worked on by a pool of host threads (the pool is
test plumbing; each call is the oracle as it stands).

On sampled tensors per model (small, medium, the largest matrix shape, a norm-gain vector)
the oracle also builds the code and the stream from the same bytes, and its stream is
compared word by word with the library's.
"""
import concurrent.futures as cf
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2505_02380_b200 as E
import workloads
from helpers import expected_out
from workloads.device import DeviceModel

pytestmark = pytest.mark.gpu


def _oracle_tensor(name, bits, w_host, q_gpu, s_gpu, z_gpu, out_gpu):
    """One tensor against the oracle; runs on a pool thread.  -> name of the first mismatch, or None."""
    q_ref, qp = oracle.quantize_tensor(w_host, bits)
    if (np.float32(qp.scale).tobytes(), qp.zero_point) != (np.float32(s_gpu).tobytes(), z_gpu):
        return f"{name}: scale / zero point"
    if not np.array_equal(q_ref, q_gpu):
        return f"{name}: symbols"
    if not np.array_equal(oracle.dequant(q_ref, qp.scale, qp.zero_point), out_gpu):
        return f"{name}: decoded fp16 output"
    return None


def _check_model(wl, sample_names):
    E.entro_set_decode_config(*E.DEFAULT_DECODE_CONFIG)
    model = DeviceModel(wl, E, E.DEFAULT_DECODE_CONFIG[0], keep_q=True)
    model.out.zero_()
    E.entro_decode_dequant_batched(model.descs)
    torch.cuda.synchronize()
    assert E.entro_last_device_status() == E.OK
    oracle.lib()                                   # built before the pool starts
    workers = max(1, min(16, os.cpu_count() or 1))
    failures, pending = [], []
    with cf.ThreadPoolExecutor(max_workers=workers) as pool:
        for spec, q, (s, z), out in zip(wl.tensors, model.q, model.qparams, model.out_slices):
            w_host = workloads.make_tensor(spec, "cuda").view(-1).cpu().numpy()
            pending.append(pool.submit(_oracle_tensor, spec.name, wl.bits, w_host, q.cpu().numpy(), s, z,
                                       out.cpu().numpy().view(np.uint16)))
            while len(pending) >= 2 * workers:     # bounds the host copies in flight
                failures.append(pending.pop(0).result())
        failures += [f.result() for f in pending]
    assert [f for f in failures if f] == []
    # sampled tensors: code and stream too
    by_name = {t.name: i for i, t in enumerate(wl.tensors)}
    for name in sample_names:
        i = by_name[name]
        spec = wl.tensors[i]
        w = workloads.make_tensor(spec, "cuda").view(-1).cpu().numpy()
        c = oracle.compress(w, wl.bits, wl.chunk_symbols)
        assert torch.equal(model.keep[i].stream.cpu(), torch.from_numpy(c.enc.stream.view(np.int32))), name
        assert torch.equal(model.keep[i].index.cpu(),
                           torch.from_numpy(np.concatenate([c.enc.offsets.view(np.uint8),
                                                            c.enc.sub_len.reshape(-1).view(np.uint8)]))), name
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
