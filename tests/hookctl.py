"""Test-side handle on the library's test hooks (mars_test_hook of the C ABI): forced row
splits, the single-block MMA kernel, cluster sizes of the stochastic tail, the top-k kernel's batch
shape.  conftest.py clears
all of them after every test."""
from paper_2601_15498_b200 import mars

NAMES = ("HOOK_FORCE_SPLIT", "HOOK_LMHEAD_SINGLE_BLOCK", "HOOK_STOCH_TAIL_CLUSTER", "HOOK_NO_OVERLAP",
         "HOOK_TOPK_VARIANT")


def set(name: str, value: int) -> None:
    mars.test_hook(getattr(mars, name), int(value))


def clear(name: str) -> None:
    mars.test_hook(getattr(mars, name), 0)


def clear_all() -> None:
    for n in NAMES:
        clear(n)
