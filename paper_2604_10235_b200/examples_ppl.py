"""Runs the chunk-selection kernels once on synthetic logits (the command the ncu summary under
profiles/ was taken with):  python -m paper_2604_10235_b200.examples_ppl [bf16|f32]"""
import sys

import torch

from . import binding as cc


def main() -> None:
    dtype = torch.float32 if len(sys.argv) > 1 and sys.argv[1] == "f32" else torch.bfloat16
    chunks, t, v = 32, 64, 128256
    ctx = cc.Context(0)
    gen_ = torch.Generator(device="cuda").manual_seed(7)
    sets = [torch.randn((chunks, t, v), device="cuda", generator=gen_).to(dtype) for _ in range(2)]
    tgt = torch.randint(0, v, (t,), device="cuda", dtype=torch.int32)
    nll = torch.empty((chunks, t), device="cuda")
    score = torch.empty((chunks,), device="cuda")
    chosen = torch.empty((6,), dtype=torch.int32, device="cuda")
    for _ in range(3):
        for x in sets:
            cc.cc_ppl_chunk_scores(ctx, x, tgt, nll, score)
    cc.cc_select_chunks(ctx, score, 6, chosen)
    assert ctx.poll() == 0
    print("lowest-perplexity chunks:", chosen.cpu().tolist())


if __name__ == "__main__":
    main()
