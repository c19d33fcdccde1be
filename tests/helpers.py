"""Glue shared by the GPU parity tests: moves oracle-made inputs to the device and calls
the library through its binding.  No method arithmetic lives here."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2505_02380_b200 as E


def index_bytes_np(enc: oracle.Encoded) -> np.ndarray:
    """The library's index layout: offsets (u64) then sub-block lengths (u16), as bytes."""
    return np.concatenate([enc.offsets.view(np.uint8), enc.sub_len.reshape(-1).view(np.uint8)])


def to_dev_stream(stream: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(stream.view(np.int32).copy()).cuda()


def to_dev_index(enc: oracle.Encoded) -> torch.Tensor:
    return torch.from_numpy(index_bytes_np(enc).copy()).cuda()


def codebook_from_oracle(c: oracle.Compressed) -> E.Codebook:
    return E.Codebook.from_lengths(c.lengths.tolist(), c.codes.tolist())


def gpu_decode_from_oracle_stream(c: oracle.Compressed, n: int, chunk: int) -> np.ndarray:
    """Decode the ORACLE's stream and index on the GPU.  -> fp16 bit patterns (uint16)."""
    out = E.entro_decode_dequant(to_dev_stream(c.enc.stream), to_dev_index(c.enc), n, chunk,
                                 codebook_from_oracle(c), c.qp.scale, c.qp.zero_point)
    torch.cuda.synchronize()
    return out.cpu().numpy().view(np.uint16)


def expected_out(c: oracle.Compressed) -> np.ndarray:
    """What decoding must give, by definition: the dequantised symbols."""
    return oracle.dequant(c.q, c.qp.scale, c.qp.zero_point)


def assert_status_ok():
    st = E.entro_last_device_status()
    assert st == E.OK, E.status_string(st)
