"""Child process of tests/test_oracle_mutations.py: runs the oracle's pin file once per library given on the
command line (name=path pairs), in this one process, and prints one JSON line per library with pytest's exit
code and the first failing pin.  Between runs the oracle front end is made to load the next library."""
import json
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import oracle  # noqa: E402


class FirstFailure:
    def __init__(self):
        self.nodeid = ""

    def pytest_runtest_logreport(self, report):
        if report.failed and not self.nodeid:
            self.nodeid = report.nodeid.split("::")[-1]


def main():
    pins = os.path.join(ROOT, "tests", "test_oracle_pins.py")
    for pair in sys.argv[1:]:
        name, path = pair.split("=", 1)
        os.environ["REF_ORACLE_LIB"] = path
        oracle._lib = None
        seen = FirstFailure()
        with open(os.devnull, "w") as null:
            out, sys.stdout = sys.stdout, null
            try:
                rc = int(pytest.main([pins, "-x", "-q", "-p", "no:cacheprovider", "--no-header"], plugins=[seen]))
            finally:
                sys.stdout = out
        print(json.dumps({"name": name, "rc": rc, "first": seen.nodeid}), flush=True)


if __name__ == "__main__":
    main()
