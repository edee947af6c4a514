"""The Python example of README.md runs as printed (inputs filled in where the text says so)."""
import os
import re

import pytest


@pytest.mark.gpu
def test_readme_example_runs_as_printed():
    import torch
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    text = open(os.path.join(root, "README.md")).read()
    code = re.search(r"```python\n(.*?)```", text, flags=re.S).group(1)
    marker = "# ... conf_prev"
    assert marker in code
    head, tail = code.split(marker, 1)
    tail = tail.split("\n", 1)[1]                                  # drop the rest of the placeholder line
    g = torch.Generator(device="cuda").manual_seed(0)
    env = {}
    exec(head, env)
    L, M, H, Hkv, d = env["L"], env["M"], env["H"], env["Hkv"], env["d"]
    env["conf_prev"] = torch.rand(L, device="cuda", generator=g)
    env["masked"] = torch.zeros(L, dtype=torch.uint8, device="cuda")
    env["masked"][M:] = 1
    env["Q"] = (torch.randn(L - M, H, d, device="cuda", generator=g) / d ** 0.5).to(torch.bfloat16)
    env["K"] = (torch.randn(Hkv, L, d, device="cuda", generator=g) / d ** 0.5).to(torch.bfloat16)
    env["V"] = torch.randn(Hkv, L, d, device="cuda", generator=g).to(torch.bfloat16)
    exec(tail, env)
    n = env["n_active"].item()
    assert 0 < n <= env["k"] * 9 and env["cnt"].min().item() == env["C"]
    assert torch.isfinite(env["O"][:n].float()).all() and env["O"][:n].float().abs().max().item() > 0
    env["ctx"].close()
