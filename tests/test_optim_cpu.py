"""The torch.optim front end without a GPU: it builds, keeps torch's parameter-group
conventions and has no CPU path to fall back on."""
import pytest
import torch

from paper_2601_07876_b200.optim import Novak


def test_groups_defaults_and_no_cpu_fallback():
    m = torch.nn.Sequential(torch.nn.Linear(4, 3), torch.nn.Linear(3, 2))
    opt = Novak([{"params": m[0].parameters()},
                 {"params": m[1].parameters(), "lr": 5e-4, "nesterov": "true",
                  "true_nesterov_steps": 100}], lr=2e-3, moment_dtype="bf16")
    assert isinstance(opt, torch.optim.Optimizer) and len(opt.param_groups) == 2
    assert opt.param_groups[0]["lr"] == 2e-3 and opt.param_groups[1]["lr"] == 5e-4
    assert opt.param_groups[0]["nesterov"] == "approximation"
    assert opt.param_groups[1]["true_nesterov_steps"] == 100
    assert opt.param_groups[0]["moment_dtype"] == "bf16"
    sd = opt.state_dict()                       # nothing stepped yet: no engine records
    assert sd["engines"] == [None, None] and "params" not in sd["param_groups"][0]
    opt.add_param_group({"params": [torch.nn.Parameter(torch.zeros(3))]})
    assert len(opt._engines) == 3
    m(torch.randn(5, 4)).sum().backward()
    opt.param_groups[2]["params"][0].grad = torch.zeros(3)
    with pytest.raises(ValueError):             # CPU tensors: refused, never stepped on the host
        opt.step()
    opt.zero_grad()
