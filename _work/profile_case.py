"""One attention-heavy case for profiling:

    python -m paper_2606_18394_b200.profile_case B L [layers [batch [paged]]]

runs `layers` attention calls (own KV buffers per layer) at the Qwen3-8B head shape, twice (warm-up and
measured), and prints the time per call.  batch > 1 gives every sequence the prefix length L; paged = 1 puts
the prefixes into a paged cache (page size 16) behind a shuffled page table.  Meant to be run under ncu with
-k / -c on a case of a few GB at most."""
import sys

import numpy as np
import torch

from .step import VerifyStep


def main():
    arg = lambda i, d: int(sys.argv[i]) if len(sys.argv) > i else d
    B, L, layers, batch, paged = arg(1, 256), arg(2, 16384), arg(3, 6), arg(4, 1), arg(5, 0)
    kw = {}
    if paged:
        per = (L + 16 + 15) // 16
        kw = dict(page_size=16, num_pages=batch * per + 8, max_pages=per)
    st = VerifyStep(batch=batch, layers=layers, Hq=32, Hkv=8, D=128, B=B, N=12, W=7, V=4096, max_seq_len=L, **kw)
    gen = torch.Generator(device="cuda").manual_seed(1)
    for t in (st.q, st.tree_k, st.tree_v):
        t.copy_(torch.randn(t.shape, generator=gen, device="cuda", dtype=torch.float32))
    for layer in range(layers):
        st.k_cache[layer].copy_(torch.randn(st.k_cache[layer].shape, generator=gen, device="cuda", dtype=torch.float32))
        st.v_cache[layer].copy_(torch.randn(st.v_cache[layer].shape, generator=gen, device="cuda", dtype=torch.float32))
    if paged:
        ids = np.random.default_rng(0).permutation(kw["num_pages"]).astype(np.int32)
        table = ids[:batch * kw["max_pages"]].reshape(batch, kw["max_pages"])
        st.page_table.copy_(torch.from_numpy(table).cuda())
    st.seq_len0.fill_(L)
    st.seq_len.fill_(L)
    st.logp.copy_(torch.log_softmax(torch.randn(st.logp.shape, generator=gen, device="cuda") * 3, -1))
    st.tree_build()
    torch.cuda.synchronize()
    for rep in range(2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for layer in range(layers):
            st.verify_attn(layer)
        e1.record()
        torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    print(f"B={B} L={L} batch={batch} paged={paged}: {e0.elapsed_time(e1) * 1e3 / layers:.2f} us per attention call, "
          f"{layers} layers")


if __name__ == "__main__":
    main()
