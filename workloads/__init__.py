"""Seeded synthetic input generators shared by the tests, the benchmark and the oracle's tests."""
from .generators import (ALL, LLAMA13B_SERVING, LLAMA7B_DECODE, LLAMA7B_PREFILL, LONG_CONTEXT, TOY,
                         Workload, decode_tokens, prompt_chunk, prompt_lens, scaled,
                         unit_bases, unit_directions)
from .views import unit_view, widen
