"""Host-side logic of the step runner that needs no GPU: how the linears of a step are batched."""
from paper_2511_23225_b200.workload import batch_partition


def test_every_linear_lands_in_exactly_one_batch_of_at_most_two():
    for n in range(1, 10):
        parts = batch_partition(n)
        assert [i for b in parts for i in b] == list(range(n))     # in order, each once
        assert all(1 <= len(b) <= 2 for b in parts)
        assert len(parts) == (n + 1) // 2                           # as few batches as pairs allow


def test_even_counts_pair_up_and_odd_counts_start_with_a_single_linear():
    assert batch_partition(4) == [[0, 1], [2, 3]]
    assert batch_partition(5) == [[0], [1, 2], [3, 4]]
    assert batch_partition(1) == [[0]]
