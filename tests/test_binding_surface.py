"""Every attribute that bench.py, the entry module and the tests read off a MoEContext exists on the class.

The GPU-side callers cannot run without a device, so a method removed from the binding would otherwise be
noticed only on a GPU machine.  This walks their syntax trees on the CPU instead."""
import ast
import glob
import os

from paper_2607_26444_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
# the name under which most callers hold a MoEContext; names bound to a MoEContext(...) call are added per file
CTX_NAMES = {"ctx"}
# `ctx` is also what the multi-process test calls its multiprocessing context
NOT_OURS = {"Queue", "Process"}


def _instance_attrs():
    """Names assigned as self.<name> anywhere in MoEContext (instance state set by __init__ and setters)."""
    src = open(os.path.join(ROOT, "paper_2607_26444_b200", "binding.py")).read()
    names = set()
    for node in ast.walk(ast.parse(src)):
        if isinstance(node, ast.ClassDef) and node.name == "MoEContext":
            for sub in ast.walk(node):
                if (isinstance(sub, ast.Attribute) and isinstance(sub.ctx, ast.Store)
                        and isinstance(sub.value, ast.Name) and sub.value.id == "self"):
                    names.add(sub.attr)
    return names


def _used_attrs(path):
    used = set()
    tree = ast.parse(open(path).read(), filename=path)
    names = set(CTX_NAMES)
    for node in ast.walk(tree):                                                  # x = [B.]MoEContext(...)
        if isinstance(node, ast.Assign) and isinstance(node.value, ast.Call):
            f = node.value.func
            if (f.attr if isinstance(f, ast.Attribute) else getattr(f, "id", "")) == "MoEContext":
                names |= {t.id for t in node.targets if isinstance(t, ast.Name)}
    for node in ast.walk(tree):
        if not isinstance(node, ast.Attribute):
            continue
        v = node.value
        if isinstance(v, ast.Name) and v.id in names:                      # ctx.<name>
            used.add(node.attr)
        elif isinstance(v, ast.Attribute) and v.attr == "ctx":                   # case.ctx.<name>, self.ctx.<name>
            used.add(node.attr)
    return used - NOT_OURS


def test_every_context_attribute_the_callers_use_exists():
    files = [os.path.join(ROOT, "bench.py"), os.path.join(ROOT, "__graft_entry__.py")]
    files += sorted(glob.glob(os.path.join(ROOT, "tests", "*.py")))
    have = set(dir(B.MoEContext)) | _instance_attrs()
    missing = {}
    for f in files:
        gone = sorted(_used_attrs(f) - have)
        if gone:
            missing[os.path.relpath(f, ROOT)] = gone
    assert not missing, f"MoEContext lacks attributes its callers use: {missing}"


def test_the_walk_sees_the_calls_it_is_meant_to_guard():
    used = _used_attrs(os.path.join(ROOT, "bench.py"))
    assert {"layout", "dispatch", "combine", "timeline", "timeline_spans", "sm_budget"} <= used


def test_every_binding_function_has_a_c_export_of_the_same_name():
    for name in B.EXPORTS:
        assert callable(getattr(B, name)), name
