"""The paper's named layouts (Sections 5.1, 5.2, Appendix A.1) through the library on a B200
against the CPU checker: prompts served in chunks, the cache state bit for bit, and a decode
step, on layouts whose first standard cache is not computed by layer 0 (MA-Offset), that hold
two standard caches on one block table (MA-Pairs) and whose standard layers share between
consecutive layers (MA-Successive)."""
import pytest

from synth import configs as cf

from test_gpu_chunks import run_chunked

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["MA-Offset", "MA-Pairs", "MA-Successive-3", "MA-Pairs-SlideShare", "MA-NoShare-3"])
def test_preset_layout_chunks_state_and_decode(name):
    window = 128
    lay = [(k, window if k == cf.SLIDING else 0, o) for k, _, o in cf.PAPER_VARIANTS[name]()]
    # the paper's head configuration: 12 query heads, 3 KV heads (head_dim 128 assumed)
    wl = cf.prefill_chunk().scaled(layout=lay, n_q_heads=12, n_kv_heads=3, batch=2, seq_len=0,
                                   name=f"preset_{name}")
    schedule = [[200, 150, 1], [70, 300, 40]]
    run_chunked(wl, schedule, scratch=1200, rows_per_chunk=12)
