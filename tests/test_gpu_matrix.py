"""Every switch against every mode: the kernel-selection flags crossed with batch size and sampling temperature on the
bf16 shape.  Each combination must run a few free steps without an error status, emit valid token counts and ids, keep its
state consistent, and (greedy, whatever the flags) emit the same tokens as the default build of the same mode: the flags
choose kernels, never results beyond rounding, so token streams may only part where the default run's own top-2 gap is tiny;
here they are required to agree on the first step."""
import pytest
import torch

import inputs

pytestmark = pytest.mark.gpu

FLAGS = [0, 1, 2, 4, 8, 16, 32, 128, 256, 4 | 8 | 16 | 256]


@pytest.mark.parametrize("temperature", [0.0, 0.7], ids=["greedy", "T0.7"])
@pytest.mark.parametrize("batch", [1, 3], ids=["b1", "b3"])
def test_flags_times_batch_times_temperature(batch, temperature):
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape("small_bf16")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w = inputs.make_weights(shape, seed=0, init="fan_in")
    w_gpu = {k: v.to("cuda:0") for k, v in w.items()}
    prompts = [inputs.make_prompt(shape.with_(prompt_len=n), seed=1 + i).tolist() for i, n in enumerate((48, 150, 17)[:batch])]
    K = shape.K
    first = {}
    for flags in FLAGS:
        model = Amphista(shape, topo, w_gpu, flags=flags, max_batch=batch, temperature=temperature, seed=11, max_ctx=256)
        roots = [model.prefill(p, seq=b) for b, p in enumerate(prompts)]
        tok = torch.zeros(batch, K + 1, dtype=torch.int32, device="cuda:0")
        n = torch.zeros(batch, dtype=torch.int32, device="cuda:0")
        lens = [len(p) for p in prompts]
        for step in range(3):
            model.step(tok, n)
            torch.cuda.synchronize()
            for b in range(batch):
                L = int(n[b])
                assert 1 <= L <= K + 1, (flags, step, b, L)
                ids = tok[b, :L].tolist()
                assert all(0 <= t < shape.vocab for t in ids)
                lens[b] += L
                C, root, pend = model.get_state(b)
                assert (C, pend) == (lens[b], L) and 0 <= root < shape.vocab
                if step == 0:
                    key = (b,)
                    if temperature == 0.0:
                        first.setdefault(key, (roots[b], ids))
                        assert first[key] == (roots[b], ids), f"flags {flags}: first step differs from flags {FLAGS[0]}"
        model.close()
