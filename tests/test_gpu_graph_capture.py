"""The library neither allocates nor synchronises, so its calls can be captured into a CUDA graph: a captured
prefill (tensor-core replay), decode steps, attention over the compressed cache and the attention loss, replayed,
must leave the same cache and outputs as the same calls issued directly."""
import numpy as np
import pytest
import torch

from paper_2412_16187_b200 import workloads as wl

from cases import PARITY_CASES
from parity import Case, to_dev

pytestmark = pytest.mark.gpu


def test_prefill_decode_attend_inside_a_cuda_graph():
    w = PARITY_CASES["llama3_8b_gqa"].scaled(decode_steps=4)
    dq, dk, dv = (to_dev(wl.gen_decode_inputs(w, x, 0, 4), w) for x in "qkv")
    results = []
    for use_graph in (False, True):
        case = Case(w)
        c = case.gpu
        ws = c.workspace(w.max_prompt_len)
        out = torch.zeros((w.n_seq, w.n_kv_heads * w.group_size, w.head_dim), dtype=torch.float32, device="cuda")
        loss = torch.zeros((w.n_seq, w.n_kv_heads * w.group_size), dtype=torch.float32, device="cuda")
        vic = torch.zeros((4, w.n_seq, w.n_kv_heads), dtype=torch.int32, device="cuda")
        st = torch.cuda.Stream()

        def body():
            c.prefill_compress(case.dQ, case.dK, case.dV, case.dplen, w.max_prompt_len, workspace=ws, stream=st)
            c.attention_loss(dq[0], case.dK, out=loss, stream=st)
            for i in range(4):
                c.decode_step(dq[i], dk[i], dv[i], victim_out=vic[i], stream=st)
            c.attend(dq[3], out, stream=st)

        with torch.cuda.stream(st):
            body()  # first call outside any capture (function attributes are set once per kernel)
            st.synchronize()
            c.reset(stream=st)
            if use_graph:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=st):
                    body()
                c.reset(stream=st)
                g.replay()
            else:
                body()
            st.synchronize()
        results.append([t.cpu().numpy().copy() for t in (c.codes, c.pos, c.scores, c.fill, c.next_pos, vic, out, loss,
                                                         c.k_cache.view(torch.int16), c.v_cache.view(torch.int16))])
    for a, b in zip(*results):
        assert np.array_equal(a, b)
