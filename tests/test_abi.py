"""The C-ABI library builds, loads without a GPU, and exports every function include/jot.h declares."""
import ctypes
import os
import re

from paper_2602_11133_b200 import build as jot_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "jot.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(jot_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib_path = jot_build.build()
    lib = ctypes.CDLL(lib_path)
    names = declared_functions()
    assert {"jot_init_model", "jot_denoise_step", "jot_accept_freeze", "jot_generate"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    from paper_2602_11133_b200 import jot
    assert sorted(jot.EXPORTS) == names


def test_host_side_calls_without_device_work():
    lib = ctypes.CDLL(jot_build.build())
    lib.jot_status_string.restype = ctypes.c_char_p
    assert lib.jot_status_string(0) == b"ok"
    assert b"wait" in lib.jot_status_string(-5)
    assert lib.jot_workspace_bytes(None, 1, 1) == 0
    from paper_2602_11133_b200 import jot
    cfg = jot.ModelConfig(2, 256, 4, 4, 64, 704, 4096, 4095, 10000.0, 1e-5)
    lib.jot_workspace_bytes.restype = ctypes.c_size_t
    lib.jot_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
    n1 = lib.jot_workspace_bytes(ctypes.byref(cfg), 1, 96)
    n2 = lib.jot_workspace_bytes(ctypes.byref(cfg), 2, 96)
    assert 0 < n1 < n2 and n1 % 1024 == 0
    bad = jot.ModelConfig(2, 250, 4, 4, 64, 704, 4096, 4095, 10000.0, 1e-5)
    assert lib.jot_workspace_bytes(ctypes.byref(bad), 1, 96) == 0
    # argument errors are reported before anything touches a device
    assert lib.jot_generate(None, None, 0, None, None, 1, 1, None, None, None, None, None, None) == -1
    assert lib.jot_accept_freeze(None, 0, 0, None, 1, 1, 0, 1, 1, None, None, None, None, None, None, None, 0, None) == -1


def test_lm_head_schedule_gives_every_accepted_row_count_a_chunk():
    """The LM head's split of (row blocks) x (vocabulary chunks) over the CTAs, on the host: every active-row
    count the entry points accept must get at least one vocabulary chunk per row block (zero chunks would leave
    rows without statistics), and the chunks must cover all vocabulary tiles."""
    from paper_2602_11133_b200 import jot
    for sms in (148, 132, 8, 3):
        limit = jot.max_active_rows(sms)
        assert limit == 128 * (sms - sms % 2)
        grid = min(sms, 256)
        for vocab in (4096, 126464, 152064):
            rows = sorted(set(list(range(1, 300)) + list(range(300, limit, 997)) + [limit - 1, limit]))
            for R in rows:
                if R > limit:
                    continue
                # the same choice of kernel shape as the library: 128-wide tiles up to 128 rows, 256-wide up to
                # 256 rows, CTA pairs beyond
                pair = R > 256
                bn = 128 if R <= 128 else 256
                n_vt = (vocab + bn - 1) // bn
                n_rb, n_ch = jot.lm_head_partition(R, grid & ~1 if pair else grid, n_vt, pair)
                assert n_rb == (R + 127) // 128
                assert 1 <= n_ch <= n_vt, (sms, vocab, R, n_rb, n_ch)
                units = (n_rb + 1) // 2 if pair else n_rb
                assert units * n_ch <= (grid // 2 if pair else grid)
        n_rb, n_ch = jot.lm_head_partition(limit + 128, grid & ~1, 988, True)
        assert n_ch == 0              # beyond the limit the schedule has no room: that is why the entry points refuse it


def test_new_host_side_argument_checks():
    lib = ctypes.CDLL(jot_build.build())
    from paper_2602_11133_b200 import jot
    assert lib.jot_set_sync(None, 0) == -1 and lib.jot_read_status(None, None) == -1
    assert lib.jot_lm_head_partition(10, 148, 988, 0, None, None) == -1
    # per-sequence parameter sets travel as kernel arguments: at most 64 sequences per call
    pars = (jot.Params * 65)(*[jot.Params() for _ in range(65)])
    one = ctypes.c_void_p(16)        # never dereferenced: the size check comes first
    assert lib.jot_accept_freeze(pars, 1, 0, one, 65, 8, 0, 8, 1, one, one, one, one, None, None, None, 0, None) == -2
