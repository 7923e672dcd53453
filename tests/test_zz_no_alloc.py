"""gls_draft_sample_static -- draft sampling without a caller-provided workspace.

Some users of the library run where device memory cannot be allocated at call time (a serving
step that must avoid cudaMalloc's device-wide synchronisation, a plug-in whose host owns all
device memory).  For them the library carries a fixed scratch buffer in its own image.  These
tests call that entry point through the C ABI and require the very same tokens and scores as
gls_draft_sample on the same inputs -- twice in a row with different inputs, because the buffer is
shared between calls and still holds the previous call's contents when the next one starts.

This file sorts after the other test files on purpose: a run that stops at the first failure has
then already run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2506_05632_b200 import synth

pytestmark = pytest.mark.gpu
SEED = synth.NOISE_SEED + 99


def _logits(B, K, J, V, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (3.0 * torch.randn(B, K, J, V, generator=g, device="cuda")).to(dtype)


def _compare(gls, logits, **kw):
    B, K, J, V = logits.shape
    assert gls.workspace_bytes(B, K, J, V) <= gls.static_scratch_bytes()
    want_tok, want_sc = gls.draft_sample(logits, **kw)
    tok = torch.full((B, K, J), -7, dtype=torch.int32, device="cuda")
    sc = torch.full((B, K, J), float("nan"), dtype=torch.float32, device="cuda")
    gls.draft_sample_static(logits, tok, sc, **kw)
    torch.cuda.synchronize()
    # integer outputs bit for bit; scores within the 1e-5 relative rule of the parity tests
    assert torch.equal(tok, want_tok)
    w, g = want_sc.double().cpu().numpy(), sc.double().cpu().numpy()
    assert np.all(np.abs(g - w) <= 1e-5 * np.maximum(1.0, np.abs(w)))


def test_two_calls_in_a_row_match_the_workspace_entry_point(gls):
    # several vocabulary slices per row, a ragged tail, both element types
    _compare(gls, _logits(5, 3, 2, 40001, torch.float32, 1), seed=SEED, inv_temp=0.9, pos_base=1)
    # second call: other shape, dtype, seed -- stale scratch from the first call must not matter
    _compare(gls, _logits(7, 2, 3, 9000, torch.bfloat16, 2), seed=SEED + 1, seq_base=11, spec=1)
    # and once more with the first shape, so that the buffer was last used by a different layout
    _compare(gls, _logits(5, 3, 2, 40001, torch.float32, 3), seed=SEED + 2)


def test_status_word_and_masked_rows(gls):
    logits = _logits(3, 2, 1, 3000, torch.float32, 4)
    logits[1, 1, 0, :] = float("-inf")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tok = torch.empty((3, 2, 1), dtype=torch.int32, device="cuda")
    gls.draft_sample_static(logits, tok, None, seed=SEED, status=status)
    torch.cuda.synchronize()
    want, _ = gls.draft_sample(logits, seed=SEED)
    assert torch.equal(tok, want) and int(tok[1, 1, 0]) == -1
    assert int(status.item()) & gls.DEV_EMPTY_SUPPORT


def test_problem_beyond_the_static_limit_is_refused(gls):
    # the check is on sizes only: a one-element tensor stands in for a huge batch via zero strides
    B, K, J, V = 4096, 8, 8, 152064
    assert gls.workspace_bytes(B, K, J, V) > gls.static_scratch_bytes()
    one = torch.zeros(1, 1, 1, V, device="cuda").expand(B, K, J, V)
    tok = torch.full((1,), -5, dtype=torch.int32, device="cuda")
    with pytest.raises(gls.GlsError, match="STATIC_LIMIT"):
        gls.draft_sample_static(one, tok, None, seed=SEED)
    torch.cuda.synchronize()
    assert int(tok.item()) == -5  # nothing was enqueued


def test_static_calls_leave_device_memory_as_it_is(gls):
    """The point of the entry point: once the first call on the device has resolved the built-in
    buffer's address, further calls obtain no device memory from the driver (free memory as the
    driver reports it is unchanged) nor from torch's allocator."""
    logits = _logits(4, 2, 2, 20000, torch.bfloat16, 5)
    tok = torch.empty((4, 2, 2), dtype=torch.int32, device="cuda")
    sc = torch.empty((4, 2, 2), dtype=torch.float32, device="cuda")
    gls.draft_sample_static(logits, tok, sc, seed=SEED)  # first use on this device
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for i in range(5):
        gls.draft_sample_static(logits, tok, sc, seed=SEED + i)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_allocated() == held0 and torch.cuda.memory_reserved() == reserved0


def test_index_self_check_found_nothing(gls):
    """When the library was built with its range checks (GLS_DEBUG_BOUNDS=1), no kernel that ran in
    this process -- every GPU test before this one -- addressed anything outside its arrays.
    Without the checks the entry point says so and the test has nothing to look at."""
    compiled_in, words = gls.debug_bounds()
    assert compiled_in in (0, 1)
    assert words[0] == 0, "range check violated %d times; first: site %d value %d limit %d" % tuple(words)
