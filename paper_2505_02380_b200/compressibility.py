"""Bits that Huffman coding saves on one grid per tensor against one grid per block of 32.

A synthetic analogue of the paper's Table 2 (Section 3, "Mixed Quantization Scheme"): the same
weights are quantised per tensor (entro_quantize_tensor) and per block (entro_quantize_blocks),
each tensor's codes get a Huffman code of their own, and "bits saved" is the symbol width minus
the mean code length.  The weights are seeded synthetic tensors with the shapes of the paper's
models, so the figures show the direction and rough size of the effect, not the paper's numbers
(those need the trained checkpoints).  Everything runs on the device through the library.

    python -m paper_2505_02380_b200.compressibility [--workload mistral|smollm|phi3] [--max-layers N] [--block 32]
"""
import argparse
import json

import numpy as np
import torch

import paper_2505_02380_b200 as E
import workloads


def _coded_bits(q: torch.Tensor, bits: int) -> int:
    counts = E.entro_histogram(q, bits)
    cb = E.entro_build_codebook(counts.tolist())
    return int((counts * cb.lengths().astype(np.uint64)).sum())


def bits_saved(wl, bits: int, block: int):
    """-> dict with the mean code length and the bits saved per weight for both grids."""
    n = tensor_bits = block_bits = 0
    for spec in wl.tensors:
        w = workloads.make_tensor(spec, "cuda").view(-1)
        qt, _ = E.entro_quantize_tensor(w, bits)
        qb, _, _ = E.entro_quantize_blocks(w, bits, block)
        tensor_bits += _coded_bits(qt, bits)
        block_bits += _coded_bits(qb, bits)
        n += spec.numel
    return {"bits": bits, "weights": n, "block": block,
            "tensor_grid": {"code_bits_per_weight": tensor_bits / n, "bits_saved": bits - tensor_bits / n},
            "block_grid": {"code_bits_per_weight": block_bits / n, "bits_saved": bits - block_bits / n},
            "improvement": (bits - tensor_bits / n) / max(bits - block_bits / n, 1e-9)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="mistral", choices=["mistral", "smollm", "phi3"])
    ap.add_argument("--max-layers", type=int, default=2)
    ap.add_argument("--block", type=int, default=32)
    args = ap.parse_args()
    make = {"mistral": workloads.mistral_7b, "smollm": workloads.smollm_1p7b, "phi3": workloads.phi3_mini_4k}[args.workload]
    out = {"workload": args.workload, "max_layers": args.max_layers, "data": "synthetic", "rows": []}
    for bits in (8, 4):
        wl = make(bits=bits, max_layers=args.max_layers)
        out["rows"].append(bits_saved(wl, bits, args.block))
    print(json.dumps(out))


if __name__ == "__main__":
    main()
