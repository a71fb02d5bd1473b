"""Runs one small case of a kernel a few times, for profilers (`ncu -k regex:<kernel> ...`).

    python -m paper_2605_13915_b200.profile_cases gemm_w8a16 M N K [calls]
    python -m paper_2605_13915_b200.profile_cases gemm_w4a16 M N K [calls]
    python -m paper_2605_13915_b200.profile_cases attn_gqa B L [calls]        (32 query heads, 8 KV heads, d 128)
    python -m paper_2605_13915_b200.profile_cases attn_mla B L [calls]        (64 query heads, latent d 576 / 512)
    python -m paper_2605_13915_b200.profile_cases attn_gqa16 B L [calls]      (128 query heads, 8 KV heads, d 128)
    python -m paper_2605_13915_b200.profile_cases attn_bf16 B L [calls]       (the BF16-KV comparison kernel, 32 / 8 heads)

Inputs are random tensors of the right types drawn on the device (KV caches: N(0,1) values quantized per token, as in
the benchmark); three weight / two cache buffers are rotated.  This is a driver for profilers, not part of the library's
API.
"""
import sys

import torch

from . import binding


def main(argv):
    what = argv[0]
    torch.manual_seed(0)
    if what in ("gemm_w8a16", "gemm_w4a16"):
        M, N, K = int(argv[1]), int(argv[2]), int(argv[3])
        calls = int(argv[4]) if len(argv) > 4 else 3
        x = torch.randn(M, K, device="cuda").to(torch.bfloat16)
        if what == "gemm_w8a16":
            w = [torch.randint(-127, 128, (N, K), dtype=torch.int8, device="cuda") for _ in range(3)]
            sc = torch.rand(N, device="cuda") * 0.01
            ws = binding.workspace(binding.gemm_w8a16_workspace_bytes(M, N, K))
            for i in range(calls):
                y = binding.gemm_w8a16(x, w[i % 3], sc, ws=ws)
        else:
            w = [torch.randint(0, 256, (N, K // 2), dtype=torch.uint8, device="cuda") for _ in range(3)]
            e = torch.randint(118, 124, (N, K // 32), dtype=torch.uint8, device="cuda")
            ws = binding.workspace(binding.gemm_w4a16_workspace_bytes(M, N, K))
            for i in range(calls):
                y = binding.gemm_w4a16(x, w[i % 3], e, ws=ws)
    elif what == "attn_bf16":
        B, L = int(argv[1]), int(argv[2])
        calls = int(argv[3]) if len(argv) > 3 else 3
        Hq, Hkv, D = 32, 8, 128
        T = B * L
        cu = (torch.arange(B + 1, dtype=torch.int32) * L).cuda()
        q = torch.randn(B, Hq, D, device="cuda").to(torch.bfloat16)
        k = [torch.randn(T, Hkv, D, device="cuda").to(torch.bfloat16) for _ in range(2)]
        v = [torch.randn(T, Hkv, D, device="cuda").to(torch.bfloat16) for _ in range(2)]
        for i in range(calls):
            y = binding.attn_decode_bf16kv(q, k[i % 2], v[i % 2], cu, L, D ** -0.5)
    elif what in ("attn_gqa", "attn_mla", "attn_gqa16"):
        B, L = int(argv[1]), int(argv[2])
        calls = int(argv[3]) if len(argv) > 3 else 3
        Hq, Hkv, D, Dv = {"attn_gqa": (32, 8, 128, 128), "attn_mla": (64, 1, 576, 512), "attn_gqa16": (128, 8, 128, 128)}[what]
        T = B * L
        cu = (torch.arange(B + 1, dtype=torch.int32) * L).cuda()
        q = torch.randn(B, Hq, D, device="cuda").to(torch.bfloat16)
        def cache(d):
            x = torch.randn(T, Hkv, d, device="cuda")
            s = x.abs().amax(dim=2) / 127.0
            return torch.clamp(torch.round(x / s[:, :, None]), -127, 127).to(torch.int8), s.contiguous()
        kk = [cache(D) for _ in range(2)]
        k, ks = [a for a, _ in kk], kk[0][1]
        v = vs = None
        if what != "attn_mla":
            vv = [cache(Dv) for _ in range(2)]
            v, vs = [a for a, _ in vv], vv[0][1]
        ws = binding.workspace(binding.attn_decode_int8kv_workspace_bytes(B, Hq, Hkv, D, Dv, L))
        for i in range(calls):
            y = binding.attn_decode_int8kv(q, k[i % 2], None if v is None else v[i % 2], ks, vs, cu, L, D ** -0.5, dv=Dv, ws=ws)
    else:
        raise SystemExit(__doc__)
    torch.cuda.synchronize()
    binding.last_device_status()
    print("ok", what, float(y.float().abs().mean()))


if __name__ == "__main__":
    main(sys.argv[1:])
