"""The index checks a -DCORUN_CHECKED build applies inside its kernels (csrc/checks.cuh), exercised on the host
through the C ABI: good indices pass, every kind of bad index is caught.  No GPU is involved: a bad index is
never handed to a kernel."""
import pytest


@pytest.fixture(scope="module")
def chk():
    from paper_2608_14376_b200 import build, corun

    build.build()
    L = corun.lib()
    import ctypes as C

    L.corun_debug_check_index.argtypes = [C.c_int32] + [C.c_int64] * 7
    return lambda kind, *a: L.corun_debug_check_index(kind, *(list(a) + [0] * (7 - len(a))))


def test_slot_and_position(chk):
    # (slot, n_slots, pos, max_blocks, kv_block)
    assert chk(0, 0, 64, 0, 272, 16) == 1
    assert chk(0, 63, 64, 272 * 16 - 1, 272, 16) == 1
    assert chk(0, 64, 64, 0, 272, 16) == 0            # slot beyond the table
    assert chk(0, -1, 64, 0, 272, 16) == 0
    assert chk(0, 3, 64, 272 * 16, 272, 16) == 0      # position beyond the block table's reach
    assert chk(0, 3, 64, -5, 272, 16) == 0
    assert chk(0, 3, 64, 5, 272, 0) == 0              # nonsense page size


def test_page_number(chk):
    assert chk(1, 0, 6000) == 1 and chk(1, 5999, 6000) == 1
    assert chk(1, 6000, 6000) == 0 and chk(1, -1, 6000) == 0 and chk(1, 2**40, 6000) == 0


def test_attention_item(chk):
    # (row, n_rows, kv head, n_kv, split, context, tokens per split)
    assert chk(2, 5, 64, 7, 8, 0, 1, 128) == 1
    assert chk(2, 5, 64, 7, 8, 31, 4071, 128) == 1    # split 31 starts at token 3968 < 4071
    assert chk(2, 5, 64, 7, 8, 32, 4071, 128) == 0    # starts beyond the context
    assert chk(2, 64, 64, 0, 8, 0, 10, 128) == 0 and chk(2, 0, 64, 8, 8, 0, 10, 128) == 0
    assert chk(2, 0, 64, 0, 8, -1, 10, 128) == 0 and chk(2, 0, 64, 0, 8, 0, 0, 128) == 0


def test_workspace_slot(chk):
    assert chk(3, 0, 0, 148) == 1 and chk(3, 147, 1, 148) == 1
    assert chk(3, 148, 0, 148) == 0 and chk(3, 0, 2, 148) == 0 and chk(3, -1, 0, 148) == 0


def test_unknown_kind(chk):
    from paper_2608_14376_b200 import corun

    assert chk(9, 0) == corun.EINVAL
