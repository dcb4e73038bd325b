"""Host-side pieces of the layer stream that need no GPU."""
from paper_2405_01943_b200.stream import skip_consecutive


def test_skip_consecutive_matches_the_papers_quarter_of_the_layers():
    skip = skip_consecutive(10, 20)                     # LLaMA2-70B: 80 layers, a quarter left dense from index 10
    dense = [l for l in range(80) if skip(l)]
    assert dense == list(range(10, 30)) and len(dense) == 80 // 4
    assert not skip_consecutive(0, 0)(0)
    assert [l for l in range(6) if skip_consecutive(4, 10)(l)] == [4, 5]
