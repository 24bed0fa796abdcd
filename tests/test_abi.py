"""The C-ABI library builds, loads and exports every symbol the header declares;
host-side argument checks work without a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import build as nbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    nbuild.build()
    return nb.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "np.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(np_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "np_init" in names and "np_sparse_mlp" in names and len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(nb.EXPORTED) == names
    assert nb.np_version() == 3


def test_struct_sizes_match_header():
    assert C.sizeof(nb.np_config) == 20 * 4
    assert C.sizeof(nb.np_sizes) == 11 * 8
    assert C.sizeof(nb.np_buffers) == 11 * C.sizeof(C.c_void_p) + 8
    assert C.sizeof(nb.np_delta_view) == 7 * C.sizeof(C.c_void_p)


def test_query_sizes_arithmetic(lib):
    # 7B shape: record 24 576 B (Section 3.5 / 4.3), buffers C * D * 2 per projection per layer
    cfg = nb.make_config(32, 4096, 11008, 512, 1101, 2752, staging_rows=256)
    s = nb.np_query_sizes(cfg)
    assert s.record_bytes == 24576
    assert s.w1_bytes == 512 * 4096 * 2 and s.w2_bytes == 32 * 11008 * 512 * 2
    assert s.backing_bytes == 32 * 11008 * 24576
    assert s.row_buffer_bytes == 32 * 2752 * 4096 * 2
    assert s.staging_bytes == 256 * 24576
    assert s.bitmap_bytes == 32 * 344 * 4 and s.logits_bytes == 32 * 11008 * 4
    assert s.host_lists_bytes == 2 * (16 + 32 * (8 + 2 * 2752)) * 4     # incoming rows, then speculative rows
    assert s.workspace_bytes >= s.logits_bytes + 5 * 4096 * 4 + 512 * 4
    assert s.dense_bytes == 0
    # a dense prefix of 8 layers: their records in one buffer, slot buffers for the other 24
    cfg8 = nb.make_config(32, 4096, 11008, 512, 1101, 2752, staging_rows=256, dense_layers=8)
    s8 = nb.np_query_sizes(cfg8)
    assert s8.dense_bytes == 8 * 11008 * 24576 and s8.row_buffer_bytes == 24 * 2752 * 4096 * 2


def test_dense_prefix_plan_matches_the_oracle(lib):
    from oracle import np_oracle as O
    cfg = nb.make_config(32, 4096, 11008, 512, 1101, 2752)
    rec = 24576
    fixed = 5 * 2**30
    for budget in [0, fixed, fixed + 32 * 2752 * rec, fixed + 32 * 2752 * rec + 3 * (11008 - 2752) * rec + 1,
                   fixed + 32 * 11008 * rec - 1, fixed + 32 * 11008 * rec, 2**45]:
        assert nb.np_plan_dense_prefix(cfg, budget, fixed) == O.dense_prefix_plan(32, 11008, 4096, 2752, budget, fixed)
    assert nb.np_plan_dense_prefix(cfg, fixed + 32 * 2752 * rec, fixed) == 0
    assert nb.np_plan_dense_prefix(cfg, fixed + 32 * 2752 * rec - 1, fixed) == -1


@pytest.mark.parametrize("field,value", [
    ("n_layers", 0), ("d_model", 100), ("d_ffn", 1000), ("d_pred", 7), ("top_k", 9999), ("capacity", 0),
    ("capacity", 99999), ("max_batch", 17), ("evict_policy", 5), ("transfer_mode", 9), ("staging_rows", 0),
    ("flags", 256), ("store_layers", -1), ("store_layers", 3), ("spec_rows", -1), ("spec_rows", 206), ("reserved", 1), ("dense_layers", -1), ("dense_layers", 3), ("io_depth", -2), ("io_depth", 5000),
])
def test_bad_config_is_rejected(lib, field, value):
    cfg = nb.make_config(2, 256, 1024, 64, 102, 205)
    setattr(cfg, field, value)
    with pytest.raises(nb.NpError) as e:
        nb.np_query_sizes(cfg)
    assert e.value.code == nb.NP_E_INVAL
    assert nb.np_last_error(None)


def test_aliased_store_is_sized_by_its_own_layers(lib):
    cfg = nb.make_config(8, 256, 1024, 64, 102, 205, store_layers=3)
    full = nb.np_query_sizes(nb.make_config(8, 256, 1024, 64, 102, 205))
    sz = nb.np_query_sizes(cfg)
    assert sz.backing_bytes * 8 == full.backing_bytes * 3 and sz.row_buffer_bytes == full.row_buffer_bytes


def test_batches_whose_hidden_vectors_do_not_fit_are_rejected(lib):
    """Sixteen sequences of 4096 hidden values need 256 KB beside the ring of the plain-core
    predictor kernel: refused at configuration time, not at the first np_predict."""
    cfg = nb.make_config(2, 256, 1024, 4096, 102, 205, max_batch=16, flags=nb.NP_F_NO_TENSOR_CORES)
    with pytest.raises(nb.NpError) as e:
        nb.np_query_sizes(cfg)
    assert e.value.code == nb.NP_E_INVAL and "do not fit" in str(e.value)
    cfg.flags = 0                                    # the tensor-core kernel takes B > 4; the ring sees at most 4
    nb.np_query_sizes(cfg)
    cfg.flags = nb.NP_F_NO_TENSOR_CORES
    cfg.max_batch = 4
    nb.np_query_sizes(cfg)
    cfg.max_batch, cfg.d_pred = 16, 2048             # 128 KB of hidden vectors + two 32 KB stages
    nb.np_query_sizes(cfg)


def test_file_mode_config_rules(lib):
    cfg = nb.make_config(2, 256, 1024, 64, 102, 205, transfer_mode=nb.NP_XFER_FILE, io_depth=256)
    assert nb.np_query_sizes(cfg).record_bytes == 1536
    cfg.record_format = nb.NP_REC_INT8               # records of 3*D + 16 bytes do not suit direct reads
    with pytest.raises(nb.NpError) as e:
        nb.np_query_sizes(cfg)
    assert e.value.code == nb.NP_E_INVAL
    cfg.record_format = nb.NP_REC_BF16
    cfg.staging_rows = 1
    with pytest.raises(nb.NpError):
        nb.np_query_sizes(cfg)


def test_null_arguments_are_rejected(lib):
    cfg = nb.make_config(2, 256, 1024, 64, 102, 205)
    bufs = nb.np_buffers()          # all NULL
    with pytest.raises(nb.NpError) as e:
        nb.np_init(cfg, bufs)
    assert e.value.code == nb.NP_E_INVAL and "NULL" in str(e.value)
    assert lib.np_predict(None, None, 1, None, None, None) == nb.NP_E_INVAL
    assert lib.np_delta(None, None, None) == nb.NP_E_INVAL
    assert lib.np_install(None, 0, 1, None) == nb.NP_E_INVAL
    assert lib.np_sparse_mlp(None, 0, None, 1, None, None) == nb.NP_E_INVAL
    assert lib.np_destroy(None) == nb.NP_OK


def test_misaligned_buffers_are_rejected(lib):
    cfg = nb.make_config(2, 256, 1024, 64, 102, 205)
    bufs = nb.np_buffers()
    for name, _ in nb.np_buffers._fields_:
        setattr(bufs, name, 0x1000)
    bufs.workspace = 0x1010
    with pytest.raises(nb.NpError) as e:
        nb.np_init(cfg, bufs)
    assert e.value.code == nb.NP_E_INVAL and "aligned" in str(e.value)
