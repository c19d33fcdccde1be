"""The file of entropy-coded weights: what is written is what is read (CPU), and a model
compressed, saved, loaded and decoded on the device equals the oracle's decode (GPU)."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from paper_2505_02380_b200 import container
from helpers import index_bytes_np


def _from_oracle(name, shape, w_np, bits, chunk):
    c = oracle.compress(w_np, bits, chunk)
    stream = torch.from_numpy(c.enc.stream.view(np.int32).copy())
    index = torch.from_numpy(index_bytes_np(c.enc).copy())
    t = container.CompressedTensor(name, shape, bits, chunk, c.qp.scale, c.qp.zero_point, c.lengths.tolist(), stream,
                                   index, int(c.enc.offsets[-1]))
    return c, t


def test_file_round_trip_on_the_host(tmp_path):
    specs = [("a.weight", (64, 96), 8, 4096, 1), ("b.gain", (100,), 8, 4096, 2), ("c.weight", (3, 5000), 4, 8192, 3)]
    tensors = []
    for name, shape, bits, chunk, seed in specs:
        w = workloads.make_values(int(np.prod(shape)), 0.02, seed).numpy()
        tensors.append(_from_oracle(name, shape, w, bits, chunk)[1])
    model = container.CompressedModel(tensors)
    path = str(tmp_path / "m.entro")
    model.save(path)
    back = container.CompressedModel.load(path, pin=False)
    assert len(back.tensors) == len(tensors)
    for a, b in zip(tensors, back.tensors):
        assert (a.name, a.shape, a.bits, a.chunk_symbols, a.zero_point, a.lengths, a.total_bits) == \
               (b.name, b.shape, b.bits, b.chunk_symbols, b.zero_point, b.lengths, b.total_bits)
        assert np.float32(a.scale) == np.float32(b.scale)
        assert torch.equal(a.stream, b.stream) and torch.equal(a.index, b.index)
    rep = back.report()
    assert rep["weights"] == sum(int(np.prod(s[1])) for s in specs)
    assert rep["coded_bytes"] < rep["quantised_bytes"] + sum(t.index.numel() for t in tensors)
    with open(path, "r+b") as f:
        f.write(b"XXXXXXXX")
    with pytest.raises(ValueError):
        container.CompressedModel.load(path, pin=False)


def _doctored(tmp_path, change):
    """A valid one-tensor file whose header entry has been changed by `change`."""
    import json
    import struct
    w = workloads.make_values(3 * 5000, 0.02, 9).numpy()
    model = container.CompressedModel([_from_oracle("w", (3, 5000), w, 8, 4096)[1]])
    path = str(tmp_path / "d.entro")
    model.save(path)
    raw = open(path, "rb").read()
    (hlen,) = struct.unpack("<Q", raw[8:16])
    head = json.loads(raw[16:16 + hlen].decode())
    change(head["tensors"][0])
    new = json.dumps(head).encode()
    start_old = (16 + hlen + container.ALIGN - 1) // container.ALIGN * container.ALIGN
    start_new = (16 + len(new) + container.ALIGN - 1) // container.ALIGN * container.ALIGN
    with open(path, "wb") as f:
        f.write(raw[:8] + struct.pack("<Q", len(new)) + new)
        f.seek(start_new)
        f.write(raw[start_old:])
    return path


@pytest.mark.parametrize("change", [
    lambda e: e.__setitem__("shape", [30, 5000]),            # more chunks than the index holds
    lambda e: e.__setitem__("chunk_symbols", 1024),          # likewise
    lambda e: e.__setitem__("chunk_symbols", 4100),          # not a multiple of 32
    lambda e: e.__setitem__("total_bits", 10 ** 9),          # more bits than the stream holds
    lambda e: e.__setitem__("bits", 5),
    lambda e: e.__setitem__("lengths", [1] * 300),
    lambda e: e.__setitem__("lengths", [40, 1]),
    lambda e: e.__setitem__("zero_point", 256),
    lambda e: e["index"].__setitem__(1, e["index"][1] - 64),  # a truncated index blob
])
def test_inconsistent_header_is_refused_on_load(tmp_path, change):
    """The decoder trusts the index to have the size that shape and chunk size imply; a file
    whose header says otherwise must not get as far as the device."""
    path = _doctored(tmp_path, change)
    with pytest.raises(ValueError):
        container.CompressedModel.load(path, pin=False)


def test_consistent_header_loads(tmp_path):
    path = _doctored(tmp_path, lambda e: None)
    assert container.CompressedModel.load(path, pin=False).tensors[0].shape == (3, 5000)


@pytest.mark.gpu
@pytest.mark.parametrize("bits", [8, 4])
def test_compress_save_load_decode_matches_oracle(tmp_path, bits):
    shapes = {"embed": (300, 256), "layers.0.q": (256, 256), "layers.0.norm": (256,), "layers.0.up": (512, 256),
              "tiny": (7,)}
    named, refs = {}, {}
    for k, (name, shape) in enumerate(shapes.items()):
        kind = "gain" if len(shape) == 1 else "matrix"
        w = workloads.make_values(int(np.prod(shape)), 0.02, 500 + k, kind)
        named[name] = w.view(shape).cuda()
        c = oracle.compress(w.numpy(), bits, 4096 if bits == 8 else 8192)
        refs[name] = oracle.dequant(c.q, c.qp.scale, c.qp.zero_point)
    model = container.compress(named, bits)
    path = str(tmp_path / "m.entro")
    model.save(path)
    loaded = container.CompressedModel.load(path)
    out = loaded.to_device()
    assert set(out) == set(shapes)
    for name, shape in shapes.items():
        assert tuple(out[name].shape) == shape
        assert np.array_equal(out[name].cpu().numpy().view(np.uint16).ravel(), refs[name]), name
    rep = loaded.report()
    assert rep["coded_bytes"] < rep["fp16_bytes"]
