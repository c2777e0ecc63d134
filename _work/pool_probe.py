"""Run cconv_pool_forward a few times on one shape (random bf16 Image): the command the pooling
profiles under ``profiles/`` were captured with.

    python -m paper_1802_06905_b200.pool_probe B,C,K,W,H,R,S,sw,sh avg|max [launches]
"""
from __future__ import annotations

import sys


def main(argv=None) -> int:
    import torch
    from . import binding
    argv = sys.argv[1:] if argv is None else argv
    B, C, K, W, H, R, S, sw, sh = (int(x) for x in argv[0].split(","))
    op = binding.POOL_MAX if argv[1] == "max" else binding.POOL_AVG
    launches = int(argv[2]) if len(argv) > 2 else 3
    Wi, Hi = sw * (W - 1) + R, sh * (H - 1) + S
    gen = torch.Generator(device="cpu").manual_seed(0x18020690 + 61)
    image = torch.randn((Wi, Hi, C, B), generator=gen).to(torch.bfloat16).cuda()
    out = torch.empty((K, H, W, B), dtype=torch.bfloat16, device="cuda")
    for _ in range(launches):
        binding.pool_forward(image, out, B, C, K, W, H, R, S, sw, sh, op=op)
    torch.cuda.synchronize()
    print("ok", float(out.float().abs().max()))
    return 0


if __name__ == "__main__":
    sys.exit(main())
