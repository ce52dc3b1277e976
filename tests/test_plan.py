"""Host logic of the streaming kernel's planner, through the C ABI's mamba_spec_describe_plan (no GPU needed):
which shapes it takes, and the invariant that keeps its rings from starving."""
import re

import pytest


@pytest.fixture(scope="module")
def binding():
    from paper_2408_15237_b200 import binding as b
    return b


B200 = dict(sm_count=148, smem_per_block=232448)


def cfg(b, **kw):
    base = dict(batch_max=1024, n_layers=1, n_heads=32, head_dim=128, d_state=128, n_groups_b=8, n_groups_c=32, conv_width=4,
                k_max=4, act_dtype=b.DTYPE_BF16, flags=b.FLAG_GATE | b.FLAG_CONV_SILU, device=0, kernel_select=b.KERNEL_AUTO)
    base.update(kw)
    return b.Config(*[base[n] for n, _ in b.Config._fields_])


def fields(text):
    return {k: int(v) for k, v in re.findall(r"(\w+)=(\d+)", text)}


def test_benchmark_shape_gets_the_streaming_kernel(binding):
    plan = binding.mamba_spec_describe_plan(cfg(binding), 16, 8, 4, **B200)
    f = fields(plan)
    assert plan.startswith("stream<") and f["N"] == 128 and f["CR"] == 64 and f["grid"] == 148 and f["groups"] == 3


@pytest.mark.parametrize("over,why", [(dict(act_dtype=0), "bf16"), (dict(conv_width=3), "conv width"), (dict(d_state=96), "state dim"),
                                      (dict(head_dim=48), "head dim"), (dict(n_heads=4, n_groups_b=1, n_groups_c=1), "head count"),
                                      (dict(flags=1 | 2 | 16), "Mamba-1")])
def test_shapes_outside_the_streaming_kernel_fall_to_the_generic_one(binding, over, why):
    c = cfg(binding, **over)
    plan = binding.mamba_spec_describe_plan(c, 16, 2 * c.k_max, c.k_max, **B200)
    assert plan.startswith("generic (") and why in plan


def test_ring_invariant_over_the_supported_shapes(binding):
    """A compute group hands back a stage with a pending store only when it starts its next chunk; the producer
    requests that chunk's inputs only once it holds the stage (or `lead` chunks earlier).  So the plan must keep
    groups <= S + lead whenever a CTA reuses stages, every group needs a raw stage plus one being filled, and
    the grid never exceeds the chunks."""
    seen = 0
    for N in (64, 128):
        for P in (32, 64, 96, 128, 256):
            for H in (8, 32, 64):
                for k_max in (1, 2, 4, 8):
                    for batch in (1, 3, 16, 64, 500):
                        for snap in (0, 8):
                            c = cfg(binding, n_heads=H, head_dim=P, d_state=N, n_groups_b=H // 8, n_groups_c=H, k_max=k_max,
                                    flags=3 | snap)
                            for k in {0, 1, k_max}:
                                plan = binding.mamba_spec_describe_plan(c, batch, 2 * k_max, k, **B200)
                                if not plan.startswith("stream<"):
                                    continue
                                f = fields(plan)
                                cr = f["CR"]
                                chunks = batch * H * (P // cr)
                                per_cta = -(-chunks // f["grid"])
                                assert 1 <= f["grid"] <= min(148, chunks)
                                assert f["R"] >= f["groups"] + 1 and 2 <= f["S"] <= 8 and 1 <= f["groups"] <= 3
                                assert f["groups"] <= f["S"] + f["lead"] or per_cta <= f["S"], plan
                                assert f["lead"] <= f["R"] - 1
                                seen += 1
    assert seen > 500


def test_a_small_shared_memory_budget_is_refused_not_overrun(binding):
    plan = binding.mamba_spec_describe_plan(cfg(binding), 16, 8, 4, sm_count=148, smem_per_block=48 * 1024)
    assert plan.startswith("generic (") and "shared memory" in plan


@pytest.mark.parametrize("k_max,t_max,k,launches,pending_only", [(12, 24, 12, 2, 1), (20, 28, 20, 2, 0), (20, 40, 20, 4, 2),
                                                                  (32, 32, 32, 2, 0), (20, 28, 0, 3, 2)])
def test_long_token_blocks_are_split_into_streaming_launches(binding, k_max, t_max, k, launches, pending_only):
    """More than 16 token rows (or more than 8 pending ones): launches that replay 8 pending rows each, then the rest in
    pieces of at most 16 rows; the first of those is planned like any call of its shape."""
    plan = binding.mamba_spec_describe_plan(cfg(binding, k_max=k_max), 16, t_max, k, **B200)
    f = fields(plan)
    assert plan.startswith("split(") and "stream<" in plan, plan
    assert f["launches"] == launches and f["pending_only"] == pending_only
    assert f["TCAP"] <= 16


def test_long_token_blocks_stay_whole_where_the_streaming_kernel_would_not_take_the_pieces(binding):
    for over in (dict(flags=1 | 2 | 16), dict(flags=1 | 2 | 8 | 64), dict(kernel_select=1), dict(act_dtype=0)):
        plan = binding.mamba_spec_describe_plan(cfg(binding, k_max=20, **over), 16, 40, 20, **B200)
        assert plan.startswith("generic ("), plan
