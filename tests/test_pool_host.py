"""Host-side logic of the speculation cache (Sec. 4.2, Eq. 2): the slot arithmetic, without a GPU."""
import pytest

from oracle import spatial_pool as sp


@pytest.mark.parametrize("IW,VSD", [(1, 1), (4, 2), (5, 3), (32, 2), (7, 8)])
def test_live_predictions_never_share_a_slot(IW, VSD):
    """Brute force over a raster scan with a step at every position: at any moment the predictions whose
    target is still ahead occupy distinct slots, all inside [0, IW * VSD * (VSD + 1) / 2), and together
    they fill the buffer exactly once the scan is VSD rows deep."""
    import paper_2510_25739_b200 as hawk
    slots = hawk.spec_cache_slots(IW, VSD)
    assert slots == sp.spec_cache_size(IW, VSD)
    made = []
    for T in range(IW * (2 * VSD + 2)):
        made += [(T, d) for d in range(1, VSD + 1)]
        live = [(p, d) for (p, d) in made if p + IW * d > T]
        made = live
        used = [hawk.spec_cache_slot(IW, VSD, p, d) for (p, d) in live]
        assert all(0 <= s < slots for s in used)
        assert len(set(used)) == len(used)
        if T >= IW * VSD:
            assert len(used) == slots


def test_overwritten_prediction_was_already_consumed():
    """The prediction that next lands in a slot is made exactly where the previous one pointed: at the
    earliest, the step that overwrites (P, d) starts at P + IW * d, the position (P, d) was made for."""
    import paper_2510_25739_b200 as hawk
    IW, VSD = 6, 4
    for d in range(1, VSD + 1):
        for P in range(IW * 3):
            s = hawk.spec_cache_slot(IW, VSD, P, d)
            later = [Q for Q in range(P + 1, P + IW * (VSD + 2)) if hawk.spec_cache_slot(IW, VSD, Q, d) == s]
            assert later and later[0] == P + IW * d
            for d2 in range(1, VSD + 1):
                if d2 != d:
                    assert all(hawk.spec_cache_slot(IW, VSD, Q, d2) != s for Q in range(IW * (VSD + 3)))
