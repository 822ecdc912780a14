"""One attention-heavy case for profiling: `python -m paper_2606_18394_b200.profile_case B L [layers]`
runs `layers` attention calls (own KV buffers per layer) of a single sequence at the Qwen3-8B head shape,
twice (warm-up and measured), and prints the time per call.  Meant to be run under ncu with -k / -c."""
import sys

import torch

from .step import VerifyStep


def main():
    B = int(sys.argv[1]) if len(sys.argv) > 1 else 256
    L = int(sys.argv[2]) if len(sys.argv) > 2 else 16384
    layers = int(sys.argv[3]) if len(sys.argv) > 3 else 6
    st = VerifyStep(batch=1, layers=layers, Hq=32, Hkv=8, D=128, B=B, N=12, W=7, V=4096, max_seq_len=L)
    gen = torch.Generator(device="cuda").manual_seed(1)
    for t in (st.q, st.tree_k, st.tree_v, st.k_cache, st.v_cache):
        t.copy_(torch.randn(t.shape, generator=gen, device="cuda", dtype=torch.float32))
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
    print(f"B={B} L={L}: {e0.elapsed_time(e1) * 1e3 / layers:.2f} us per attention call, {layers} layers")


if __name__ == "__main__":
    main()
