"""Builds and runs the instruction issue-rate microbenchmark (csrc/issue_rates.cu) on GPU 0 and prints its table:

    python -m paper_2609_05419_b200.issue_rates
"""
import subprocess
import sys

from . import build


def main() -> int:
    return subprocess.run([build.build_issue_rates()]).returncode


if __name__ == "__main__":
    sys.exit(main())
