"""The optional CTA shape of the tcgen05 path whose two query tiles share one K/V ring
(ORTHRUS_TC_ROW_TILES_PER_CTA=2) is chosen when the library is first used in a process, so its
parity run happens in a child process: the shape, split and in-cache tests with the variable set
(they include units of 256 rows and more, with odd numbers of query tiles)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def test_parity_with_two_query_tiles_per_cta():
    env = dict(os.environ, ORTHRUS_TC_ROW_TILES_PER_CTA="2")
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(HERE, "test_gpu_attend.py"),
                        os.path.join(HERE, "test_gpu_truncate_commit.py"), "-x", "-q",
                        "-k", "tcgen05 and (shapes or forced or peaked or cache)"],
                       env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
