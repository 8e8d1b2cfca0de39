"""Units of at most 64 query rows run, by default, the form of the tcgen05 kernel that passes the
probabilities through shared memory and issues the two products from two warps; the default parity
tests therefore cover that form.  The common form must keep serving such units too
(ORTHRUS_TC_SMALL_ROWS=0, read when the library is first used in a process): its parity run happens
in a child process, on the shape, split, edge-case and in-cache tests."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def test_parity_of_the_common_form_on_units_of_at_most_64_rows():
    env = dict(os.environ, ORTHRUS_TC_SMALL_ROWS="0")
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(HERE, "test_gpu_attend.py"),
                        os.path.join(HERE, "test_gpu_attend_tc_edges.py"),
                        os.path.join(HERE, "test_gpu_truncate_commit.py"), "-x", "-q",
                        "-k", "tcgen05 or edges or cache"],
                       env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
