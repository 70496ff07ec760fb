"""Workload shapes used by the parity tests: the five configurations, reduced where the CPU oracle would
otherwise need minutes. Reduced cases keep the dtype, hash width, group size, key structure and a budget
that is not a multiple of any tile size, so they still span several tiles and a ragged tail."""
from paper_2412_16187_b200 import workloads as wl

C = wl.CONFIGS

PARITY_CASES = {
    # full size
    "tiny": C["tiny"],
    # all 32 heads, shorter prompt
    "llama2_7b_layer": C["llama2_7b_layer"].scaled(prompt_len=1536, budget=777, decode_steps=48),
    # 3 of 16 sequences, shorter prompt, budget with a ragged tail
    "llama3_8b_gqa": C["llama3_8b_gqa"].scaled(batch=3, prompt_len=2048, budget=1000, decode_steps=40),
    # 2 of 32 layers, 30 % budget of a 4096-token prompt
    "long_prefill": C["long_prefill"].scaled(layers=2, prompt_len=4096, budget=1228, decode_steps=24),
    # 5 of 64 sequences, ragged budgets in [96, 700], prompts twice the budget
    "throughput_batch": C["throughput_batch"].scaled(batch=5, budget_lo=96, budget_hi=700, decode_steps=32),
    # the paper's protected windows (first 4, newest 10) on a GQA shape
    "protected_gqa": C["llama3_8b_gqa"].scaled(batch=2, prompt_len=700, budget=301, decode_steps=40, n_sink=4, n_recent=10),
    "protected_tiny": C["tiny"].scaled(n_sink=4, n_recent=10),
}
