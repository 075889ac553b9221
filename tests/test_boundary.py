"""The C-ABI library loads and exports every symbol include/ampnet.h declares (no compute calls: no GPU here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1705_09786_b200 import build
    build.build()                       # nvcc cross-compiles for sm_100a without a GPU
    from paper_1705_09786_b200 import load_library
    return load_library()


def declared_functions():
    src = open(os.path.join(ROOT, "include", "ampnet.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = set(re.findall(r"\b(ampnet_[a-z_]+)\s*\(", src))
    return sorted(n for n in names if not n.endswith("_fn"))


def test_every_declared_entry_point_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ampnet.h but not exported"
    from paper_1705_09786_b200.binding import EXPORTS
    assert sorted(EXPORTS) == names


def test_enum_codes_agree_with_the_input_module():
    """The integer codes of the IR format are written three times (header, oracle, input module)."""
    from workloads import ir
    src = open(os.path.join(ROOT, "include", "ampnet.h")).read()
    codes = {k: int(v) for k, v in re.findall(r"\bAMPNET_([A-Z_0-9]+)\s*=\s*(\d+)", src)}
    pairs = {"SOURCE": ir.SOURCE, "LINEAR": ir.LINEAR, "LOOKUP": ir.LOOKUP, "GRUCELL": ir.GRUCELL, "LOSS_CE": ir.LOSS_CE,
             "LOSS_MSE": ir.LOSS_MSE, "NPT_SUMROWS": ir.NPT_SUMROWS, "COND": ir.COND, "PHI": ir.PHI, "ISU": ir.ISU,
             "CONCAT": ir.CONCAT, "SPLIT": ir.SPLIT, "BCAST": ir.BCAST, "GROUP": ir.GROUP, "UNGROUP": ir.UNGROUP,
             "FLATMAP": ir.FLATMAP, "SINK": ir.SINK, "NPT_LSTM": ir.NPT_LSTM, "LSTM_LEAF": ir.LSTM_LEAF, "LSTM_BRANCH": ir.LSTM_BRANCH, "ACT_TANH": ir.ACT_TANH, "ACT_SIGMOID": ir.ACT_SIGMOID,
             "SRC_GRAPH_NODES": ir.SRC_GRAPH_NODES, "SRC_TREE_LEAVES": ir.SRC_TREE_LEAVES,
             "SRC_TREE_LEAVES_GROUPED": ir.SRC_TREE_LEAVES_GROUPED, "UNGROUP_LEAVES": ir.UNGROUP_LEAVES,
             "COND_IT_LT": ir.COND_IT_LT, "COND_BY_U": ir.COND_BY_U, "COND_ROUND_ROBIN": ir.COND_ROUND_ROBIN, "ISU_TREE_PARENT": ir.ISU_TREE_PARENT,
             "ISU_IT_INC": ir.ISU_IT_INC, "CONCAT_BY_STATE_PORT": ir.CONCAT_BY_STATE_PORT,
             "GROUP_ALL_NODES": ir.GROUP_ALL_NODES, "GROUP_EDGES_BY_DST": ir.GROUP_EDGES_BY_DST,
             "UNGROUP_TYPE_EDGES": ir.UNGROUP_TYPE_EDGES, "FLATMAP_OUT_EDGES": ir.FLATMAP_OUT_EDGES,
             "LABEL_PER_TREE_NODE": ir.LABEL_PER_TREE_NODE, "KIND_TYPED_GRAPHS": ir.KIND_TYPED_GRAPHS,
             "KIND_BINARY_TREES": ir.KIND_BINARY_TREES, "FLAG_SOURCE_ADJACENT": ir.FLAG_SOURCE_ADJACENT}
    for k, v in pairs.items():
        assert codes[k] == v, k


def test_product_fails_loudly_without_a_device(lib):
    """No CPU fallback: without a CUDA device the engine refuses to start."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    import paper_1705_09786_b200 as amp
    from workloads import ir
    with pytest.raises(RuntimeError):
        amp.Engine(ir.mlp((4, 3, 2)))
    out = ctypes.c_void_p()
    from paper_1705_09786_b200.binding import IRDesc
    import numpy as np
    g = ir.mlp((4, 3, 2))
    nodes, edges = np.ascontiguousarray(g.nodes), np.ascontiguousarray(g.edges)
    desc = IRDesc(len(nodes), len(edges), nodes.ctypes.data, edges.ctypes.data, 0)
    rc = lib.ampnet_graph_create(ctypes.byref(desc), 1, None, None, ctypes.byref(out))
    assert rc == 3 and not out.value        # AMPNET_ECUDA, no handle


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_1705_09786_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"


def test_library_ir_builders_emit_the_canonical_graphs(lib):
    """The host IR builders of the library and the tables of the shared input module describe the same graphs."""
    import numpy as np
    import paper_1705_09786_b200 as amp
    from workloads import ir
    cases = [("mlp", ([784, 256, 256, 10],), ir.mlp()), ("mlp", ([5, 3],), ir.mlp((5, 3))),
             ("rnn", (14, 128, 128, 10, ir.ACT_TANH), ir.rnn()), ("tree", (20000, 300, 150, 5), ir.tree()), ("tree_grouped", (20000, 300, 150, 5), ir.tree(grouped_leaves=True)),
             ("tree_lstm", (20000, 300, 150, 5), ir.tree_lstm()),
             ("rnn_replicated", (14, 128, 128, 10, ir.ACT_TANH, 1), ir.rnn()),
             ("rnn_replicated", (14, 16, 16, 10, ir.ACT_TANH, 3), ir.rnn(14, 16, 16, 10, replicas=3)),
             ("ggnn", (15, 100, 4, 4, 100), ir.ggnn()), ("ggnn", (7, 8, 2, 3, 5), ir.ggnn(7, 8, 2, 3, 5))]
    for family, args, want in cases:
        nodes, edges = amp.ir_tables(family, *args)
        np.testing.assert_array_equal(nodes, want.nodes)
        np.testing.assert_array_equal(edges, want.edges)
    with pytest.raises(amp.AmpnetError):
        amp.ir_tables("rnn", 14, 64, 128, 10, ir.ACT_TANH)       # Concat ports need one common width
    with pytest.raises(amp.AmpnetError):
        amp.ir_tables("mlp", [784])
