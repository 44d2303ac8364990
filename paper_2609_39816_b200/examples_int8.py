"""Small runnable example (also the command profiled in profiles/int8_group_gemm_4096.md): quantise two operands with
the group quantiser and run the classical int8 operator on them.

    python -m paper_2609_39816_b200.examples_int8 [M K N]
"""
import sys

import torch

from . import binding as lib


def main(argv):
    M, K, N = (int(x) for x in argv[1:4]) if len(argv) >= 4 else (4096, 4096, 4096)
    A = torch.randn(M, K, device="cuda")
    B = torch.randn(N, K, device="cuda") * 0.02
    cA = torch.empty((M, K), dtype=torch.int8, device="cuda")
    dA = torch.empty((M, K // 128), dtype=torch.float32, device="cuda")
    cB = torch.empty((N, K), dtype=torch.int8, device="cuda")
    dB = torch.empty((N, K // 128), dtype=torch.float32, device="cuda")
    lib.int8_quantize(A, 31, cA, dA)
    lib.int8_quantize(B, 31, cB, dB)
    ws = torch.empty(max(lib.int8_gemm_workspace(None, M, K, N), 256), dtype=torch.uint8, device="cuda")
    C = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    for _ in range(3):
        lib.int8_gemm(None, 31, cA, dA, cB, dB, C, ws)
    torch.cuda.synchronize()
    lib.device_status(ws)
    ref = (A @ B.t()).float()
    rel = ((C.float() - ref).norm() / ref.norm()).item()
    print(f"int8 operator {M}x{K}x{N}: relative error against the fp32 product {rel:.4f}")


if __name__ == "__main__":
    main(sys.argv)
