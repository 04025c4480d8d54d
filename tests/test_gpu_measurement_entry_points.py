"""The measurement entry points of the C ABI (loopspec_time_kernel, loopspec_launches_per_step, loopspec_decode_paths):
they run, report what the header says, leave the context usable, and what they report matches what a decode step does."""
import numpy as np
import pytest

from tests import gpu_util as U
import workloads as W

pytestmark = pytest.mark.gpu


def test_decode_paths_follow_the_row_and_context_capacity():
    """Passes of up to 8 rows: mma.sync cluster kernels; 9 to 64 rows of a bf16 model: the tcgen05 kernel + epilogue;
    a context capacity beyond 2560 positions (512 when the context holds several sequences): the streaming attention kernel;
    fp32 weights never leave the CUDA cores."""
    cases = [(dict(name="tiny_bf16", max_seqs=1, max_ctx=256), (0, 0)),
             (dict(name="tiny_bf16", max_seqs=4, max_ctx=256), (1, 0)),
             (dict(name="tiny_bf16", max_seqs=1, max_ctx=3000), (0, 1)),
             (dict(name="tiny_bf16", max_seqs=4, max_ctx=1024), (1, 1)),
             (dict(name="tiny_bf16", max_seqs=4, max_ctx=512), (1, 0)),
             (dict(name="tiny_raven", max_seqs=1, max_ctx=256), (1, 0)),
             (dict(name="tiny", max_seqs=4, max_ctx=256), (0, 0))]
    for kw, want in cases:
        shape = W.CONFIGS[kw["name"]]
        d1, d2 = (2, 8) if shape.R >= 16 else (1, 2)
        ctx = U.make_ctx(kw["name"], d1, d2, max_seqs=kw["max_seqs"], max_ctx=kw["max_ctx"])
        assert ctx.decode_paths() == want, (kw, ctx.decode_paths())
        ctx.close()


def test_launch_count_matches_the_kernels_of_a_pass():
    """1 preparation + 5 kernels per block + lm_head + selection + control + KV commit for passes of up to 8 rows;
    two launches per GEMM on the tcgen05 path."""
    shape = W.CONFIGS["tiny_bf16"]
    ctx = U.make_ctx("tiny_bf16", 1, 2, max_seqs=1, max_ctx=128)
    assert ctx.launches_per_step() == 1 + 5 * shape.n_recurrent + 4
    ctx.close()
    ctx = U.make_ctx("tiny_bf16", 1, 2, max_seqs=4, max_ctx=128)
    assert ctx.launches_per_step() == 1 + 9 * shape.n_recurrent + 4
    ctx.close()


@pytest.mark.parametrize("max_ctx", [512, 3000])
def test_kernels_can_be_timed_alone_and_the_context_stays_usable(max_ctx):
    """Every kernel of the pass through loopspec_time_kernel: sane times, the byte counts of the header's formulas, and
    a decode after a new prefill still matches the oracle."""
    name = "tiny_bf16"
    shape = W.CONFIGS[name]
    ref = U.oracle_run(name, 20, 12, 1, 2, T=1.0, seed=5)
    ctx = U.make_ctx(name, 1, 2, T=1.0, seed=5, max_seqs=2, max_ctx=max_ctx, max_prefill_rows=32)
    assert ctx.prefill(ref["prompt"]) == ref["first"]
    hq, hkv = shape.n_q_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim
    wbytes = [(hq + 2 * hkv) * shape.hidden * 2, shape.hidden * hq * 2, 2 * shape.ffn * shape.hidden * 2, shape.hidden * shape.ffn * 2,
              shape.vocab * shape.hidden * 2]
    for which in range(5):
        ms, nbytes = ctx.time_kernel(which, 4, 5)
        assert 0 < ms < 5.0 and nbytes == wbytes[which]
    kv_ctx = 2 * hkv * (max_ctx - 64) * 2
    ms, nbytes = ctx.time_kernel(5, 6, 5)           # decode attention: every row a context of its own
    assert 0 < ms < 50.0 and nbytes == 6 * kv_ctx
    ms, nbytes = ctx.time_kernel(6, 32, 5)          # prefill attention: the rows share one context
    assert 0 < ms < 50.0 and nbytes == kv_ctx
    with pytest.raises(Exception):
        ctx.time_kernel(6, 33, 1)                   # more rows than a prefill pass carries
    with pytest.raises(Exception):
        ctx.decode(4)                               # the timed launches used the sequences' state: a prefill comes first
    assert ctx.prefill(ref["prompt"]) == ref["first"]
    ctx.decode(12)
    U.assert_same_run(ctx, ref, 12)
    ctx.close()
