"""Every kernel on a ragged size under the range-checking build of the library.

The box this suite runs on offers no memory checker, so the library carries its own: the build with
-DBT_BOUNDS_CHECK (tests/checking_libs.py) tests every global store of every kernel against the extent
of the buffer it belongs to, skips a store that would fall outside and counts it in a device word.
Each case below runs the parity check of one kernel family against the CPU oracle -- the very functions
of the other test files, called on sizes with a ragged tail -- with that build in place of the product
library, then reads the counter: it must be zero (and the parity check must have passed, which it could
not had a store been skipped).  Nothing here is expected to fault; a stray store would be dropped, not made.
"""
import pytest
import torch

from paper_2110_15362_b200 import binding as B
from tests import checking_libs as C
from tests import gpu_util
from tests import test_gpu_arena, test_gpu_batch, test_gpu_host_forms, test_gpu_mask, test_gpu_maxpool
from tests import test_gpu_narrow, test_gpu_parity, test_gpu_prune, test_gpu_relu6

pytestmark = pytest.mark.gpu

KINDS = ["f32", "f16", "bf16", "f64"]
RAGGED = 8192 * 150 + 4097 + 13          # more tiles than SMs for every element width, last chunk and word partial


@pytest.fixture()
def checked(monkeypatch):
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    L = C.bounds_lib()
    monkeypatch.setattr(B, "_lib", L)
    assert L.bt_test_bounds_violations(1) >= 0            # the counter is reachable; start from zero
    yield L
    torch.cuda.synchronize()
    assert L.bt_test_bounds_violations(1) == 0, "a kernel tried to store outside one of its buffers"


@pytest.mark.parametrize("kind", KINDS)
def test_compress_and_decompress(checked, oracle, kind):
    test_gpu_parity.test_compress_decompress_edge_sizes(gpu_util, oracle, kind, RAGGED)
    test_gpu_parity.test_compress_decompress_edge_sizes(gpu_util, oracle, kind, 33)
    test_gpu_parity.test_compress_decompress_sparsity_levels(gpu_util, oracle, kind, 0.99)


@pytest.mark.parametrize("kind", ["bf16", "f16"])
def test_two_byte_runs_in_16_byte_units(checked, oracle, kind):
    test_gpu_parity.test_two_byte_runs_at_every_offset_from_a_16_byte_boundary(gpu_util, oracle, kind, 5)


def test_capacity_overflow(checked, oracle):
    test_gpu_parity.test_capacity_overflow_reports_and_stays_in_bounds(gpu_util, oracle)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("mode", ["stash_only", "with_y", "in_place"])
def test_relu_forward(checked, oracle, kind, mode):
    test_gpu_parity.test_relu_fwd_compress(gpu_util, oracle, kind, RAGGED, mode)


@pytest.mark.parametrize("kind", KINDS)
def test_relu_backward(checked, oracle, kind):
    test_gpu_parity.test_relu_bwd_from_bitmap(gpu_util, oracle, kind, RAGGED, False)
    test_gpu_parity.test_relu_bwd_from_bitmap(gpu_util, oracle, kind, 7, True)


@pytest.mark.parametrize("kind", KINDS)
def test_prune(checked, oracle, kind):
    test_gpu_prune.test_prune_near_thresholds(gpu_util, oracle, kind, 0.05, 16384 * 3 + 1001, "with_y")


@pytest.mark.parametrize("to_kind", ["f16", "bf16"])
def test_narrow_and_widen(checked, oracle, to_kind):
    test_gpu_narrow.test_plain_form(gpu_util, oracle, to_kind, 16384 * 3 + 1001)
    test_gpu_narrow.test_fused_form(gpu_util, oracle, to_kind, 0.05, 16384 * 5 + 123, "with_y")
    test_gpu_narrow.test_capacity_is_counted_in_16_bit_elements(gpu_util, oracle, to_kind)


@pytest.mark.parametrize("kind", KINDS)
def test_relu6_pair(checked, oracle, kind):
    test_gpu_relu6.test_relu6_pair(gpu_util, oracle, kind, 16384 * 3 + 1001, "with_y")


@pytest.mark.parametrize("kind", KINDS)
def test_mask(checked, oracle, kind):
    test_gpu_mask.test_mask_compress_edge_sizes(gpu_util, oracle, kind, 8192 * 37 + 5, "with_y")
    test_gpu_mask.test_mask_compress_edge_sizes(gpu_util, oracle, kind, 8192 * 37 + 5, "stash_only")
    test_gpu_mask.test_capacity_below_nnz_suppresses_stores(gpu_util, oracle)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("shape", [(5, 14, 14), (37, 18, 24), (33, 112, 2), (3, 6, 40)])   # pair and vector forms
def test_maxpool(checked, oracle, kind, shape):
    test_gpu_maxpool.test_forward_and_backward_match_the_oracle(gpu_util, oracle, kind, shape)


def test_arena_forms(checked, oracle):
    test_gpu_arena.test_pushes_of_mixed_types_and_round_trip(oracle)
    test_gpu_arena.test_arena_too_small_reports_and_keeps_the_cursor(oracle)
    test_gpu_arena.test_narrowed_and_relu6_pushes_share_one_arena(oracle)


@pytest.mark.parametrize("kind", KINDS)
def test_batched_forms(checked, oracle, kind):
    test_gpu_batch.test_batch_equals_the_oracle_tensor_by_tensor(oracle, kind, False, False)
    test_gpu_batch.test_batch_equals_the_oracle_tensor_by_tensor(oracle, kind, True, True)
    test_gpu_batch.test_batched_consumers_equal_the_oracle_tensor_by_tensor(oracle, kind)
    test_gpu_batch.test_arena_batch_is_the_sequence_of_single_arena_pushes(oracle, kind, True)


def test_arena_batch_that_runs_full(checked, oracle):
    test_gpu_batch.test_arena_batch_over_several_launches_and_an_arena_that_runs_full(oracle)


def test_host_forms(checked, oracle):
    test_gpu_host_forms.test_host_round_trip_and_relu_pair(oracle, "bf16", 8192 * 5 + 123)
