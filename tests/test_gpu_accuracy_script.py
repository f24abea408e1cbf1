"""The synthetic accuracy comparison (python -m paper_2503_19950_b200.accuracy) on a short context: the orderings
that follow from the method itself must hold -- dropping the removed tokens costs several times the error of
quantising them to 2 bits (the paper's argument against eviction, Sec. 2.3), 4-bit codes are several times closer
than 2-bit codes (Table 3), and the compression ratios are those of the storage format."""
import math

import pytest

from paper_2503_19950_b200 import accuracy, build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_orderings_of_the_synthetic_accuracy_table():
    rows = accuracy.run(ctx=3072, lengths=3)
    assert len(rows) == 4 * 4 + 2                           # four shapes x four 2-bit variants, two 4-bit rows
    by = {(r["shape"], r["bits"], r["filter"]): r for r in rows}
    for r in rows:
        assert math.isfinite(r["rel_l1"]) and r["rel_l1"] > 0 and math.isfinite(r["worst_rel_max"])
    for shape in {r["shape"] for r in rows}:
        for filt in ("log (Algorithm 1)", "recent window"):
            quant = by[(shape, 2, filt)]
            evict = by[(shape, 0, filt + ", eviction" if filt.startswith("recent") else "log, eviction")]
            assert evict["rel_l1"] > 2.5 * quant["rel_l1"], (shape, filt)
            assert evict["compression"] > quant["compression"] > 3.0
            assert quant["compression"] < 16.0 / 2          # codes alone would give 8x; scale/zero and the bf16 rows cost
    for filt in ("log (Algorithm 1)", "recent window"):
        two, four = by[("Hq32/Hkv8 W128 G32", 2, filt)], by[("Hq32/Hkv8 W128 G32", 4, filt)]
        assert four["rel_l1"] < two["rel_l1"] / 3
        assert four["compression"] < two["compression"]
