"""Prints Philox4x32-10 words from Triton's own implementation, run by Triton's CPU
interpreter (an independent library routine used to pin the oracle's generator).

usage: TRITON_INTERPRET=1 python philox_triton_ref.py  -> JSON on stdout
"""
import json
import os

assert os.environ.get("TRITON_INTERPRET") == "1"

import torch  # noqa: E402
import triton  # noqa: E402
import triton.language as tl  # noqa: E402


@triton.jit
def _kernel(out_ptr, seed, c_ptr, n: tl.constexpr):
    i = tl.arange(0, n)
    c0 = tl.load(c_ptr + i)
    c1 = tl.load(c_ptr + n + i)
    c2 = tl.load(c_ptr + 2 * n + i)
    c3 = tl.load(c_ptr + 3 * n + i)
    a, b, c, d = tl.philox(seed, c0, c1, c2, c3)
    tl.store(out_ptr + i, a)
    tl.store(out_ptr + n + i, b)
    tl.store(out_ptr + 2 * n + i, c)
    tl.store(out_ptr + 3 * n + i, d)


def main():
    n = 8
    cases = []
    g = torch.Generator().manual_seed(1234)
    for seed in [0, 1, 5, 0x0123456789ABCDEF, (1 << 63) - 1]:
        ctr = torch.randint(0, 2 ** 31 - 1, (4, n), generator=g, dtype=torch.int64)
        ctr[:, 0] = 0
        ctr[0, 1] = 1
        ctr[0] = torch.arange(n)            # env index in word 0, like the sampler
        ctr[3] = 0
        c32 = ctr.to(torch.int32).contiguous()
        out = torch.zeros(4 * n, dtype=torch.int32)
        _kernel[(1,)](out, seed, c32, n)
        o = out.view(4, n).to(torch.int64) & 0xFFFFFFFF
        for j in range(n):
            cases.append({"seed": seed, "counter": [int(v) for v in ctr[:, j]],
                          "out": [int(v) for v in o[:, j]]})
    # counters of the form (i, 0, 0, 1): the stream the seeded weight initialisation draws from
    for seed in [7, 0x0123456789ABCDEF]:
        ctr = torch.zeros((4, n), dtype=torch.int64)
        ctr[0] = torch.tensor([0, 1, 2, 3, 1000, 65535, 123456, 2 ** 31 - 1])
        ctr[3] = 1
        c32 = ctr.to(torch.int32).contiguous()
        out = torch.zeros(4 * n, dtype=torch.int32)
        _kernel[(1,)](out, seed, c32, n)
        o = out.view(4, n).to(torch.int64) & 0xFFFFFFFF
        for j in range(n):
            cases.append({"seed": seed, "counter": [int(v) for v in ctr[:, j]],
                          "out": [int(v) for v in o[:, j]]})
    print(json.dumps(cases))


if __name__ == "__main__":
    main()
